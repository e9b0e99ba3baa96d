// Host side of libkurtail: argument checks, workspace carving, tensor-map
// construction and the sequencing of kernels on one stream.  See
// include/kurtail.h for the contract of every entry point.
#include <cuda.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <mutex>
#include <new>

#include "../../include/kurtail.h"
#include "elementwise.cuh"
#include "fused_small.cuh"
#include "gemm_sm100.cuh"
#include "small_orth.cuh"

namespace kt {

constexpr int kHistMax = 4096;  // loss-history slots kept on the device between host read-backs
constexpr int kIdsChunk = 256;  // kt_fit_shared: steps whose sample ids are on the device at a time
constexpr int kMaxSharedBufs = 4096;  // kt_fit_shared: activation buffers one rotation can be shared by
constexpr int kProfPairs = 8192; // CUDA-event pairs available to one profiling window
enum GemmCat : int { kCatForward = 0, kCatBackwardA = 1, kCatBackwardB = 2, kCatSquare = 3, kCatQuant = 4, kCatFused = 5 };

struct DeviceBlock {
  Scalars sc;
  double hist[kHistMax];
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Split-K plan for the token contraction dR = X^T G (M = N = d, K = tokens).  The output has only
// (d/128)*(d/BN) tiles, each walking all tokens: with few tiles (d = 128: one) most SMs would idle, and with
// 512 tiles on 148 SMs the last of 3.46 waves is mostly empty.  Cutting K into s runs gives tiles*s work units.
// s minimises a time model: (waves of units)/s tile times at ~10 TFLOP/s per SM, plus, for s > 1, the pass that
// sums the s partial outputs ((2s+1) d^2 floats of traffic at ~6 TB/s and a launch).
constexpr int kPlanSMs = 148;
struct SplitPlan {
  int splits, kb_per_split;
};
static SplitPlan plan_split_k(int64_t d, int64_t K) {
  const int bn = (d % 256 == 0) ? 256 : 128;
  const long long tiles = (d / 128) * (d / bn);
  const int k_blocks = static_cast<int>((K + 63) / 64);
  const double t_tile_us = 128.0 * bn * static_cast<double>(K) * 2.0 / 1.0e7;
  const double dd_bytes = static_cast<double>(d) * d * 4.0;
  int best = 1;
  double best_cost = 1e300;
  for (int s = 1; s <= 4 * kPlanSMs; ++s) {
    const int per = (k_blocks + s - 1) / s;
    if (s > 1 && (per < 16 || s * dd_bytes > 1073741824.0)) break;
    const long long waves = (tiles * s + kPlanSMs - 1) / kPlanSMs;
    double cost = static_cast<double>(waves) / s * t_tile_us;
    if (s > 1) cost += (2.0 * s + 1.0) * dd_bytes / 6.0e6 + 5.0;
    if (cost < best_cost * 0.98) {  // a larger s must win by 2 %
      best_cost = cost;
      best = s;
    }
  }
  SplitPlan p;
  p.kb_per_split = (k_blocks + best - 1) / best;
  p.splits = (k_blocks + p.kb_per_split - 1) / p.kb_per_split;  // every run non-empty
  return p;
}

// Where everything lives inside the caller's workspace for an (N, d) problem.
struct WsLayout {
  size_t rt_hi, rt_lo;  // R^T as bf16 hi/lo  [d][d]
  size_t r_hi, r_lo;    // R   as bf16 hi/lo  [d][d]
  size_t z_hi, z_lo;    // transposed iterate of the retraction; also dR hi (before) and E hi (after)
  size_t w_hi, w_lo;    // skew direction W as bf16
  size_t fbuf;          // d x d float32: A, then P, then R^T R, then R E
  size_t dr;            // d x d float32: gradient inside kt_fit
  size_t xb;            // dense bf16 copy of a float32 X, or of any X after RMSNorm  [N][d]
  size_t xt, gt;        // X^T and G^T as bf16  [d][ldt]
  size_t ybuf;          // Y = X R [N][d], kept by the forward pass unless the backward recomputes it: float16 with
                        // a power-of-two factor per half tile row (backward_mode 0) or float32 (backward_mode 2)
  size_t yexp;          // [P][N] bytes: the exponents of those factors
  size_t partial;       // [P][N] float4 partial moment records
  size_t coef, moments; // [N] float4 each
  size_t block_loss, block_deg, norm_blocks;
  size_t rowmax, rowmin, qerr;  // quantizer: [N] uint each, [P][N] float
  size_t colpart;       // [d/32][d] float: column sums of squares of R by row slab
  size_t diag;          // [d] float: exact diagonal of R^T R - I
  size_t pvec;          // [2][d] float: the last two vectors of the power iteration on W
  size_t splitk;        // [splits][d][d] float: partial dR of the split-K backward-B (when splits > 1)
  size_t small;         // d <= 512: scratch of the one-launch orthogonal step (6 d x d floats + per-CTA partials)
  size_t adam_m;        // d x d float32: momentum of Cayley Adam inside kt_fit (only when asked for)
  size_t gather_ids;    // kt_fit_shared: [kIdsChunk][batch] int sample ids
  size_t gather_bases;  // kt_fit_shared: [kMaxSharedBufs] buffer base pointers
  size_t flat;          // flattened-kurtosis mode: the global coefficients, the global mean, 3 x [blocks] doubles
  size_t rowscale;      // [N] float: RMSNorm factor of every row (kt_config.rmsnorm), or, for the single-pass
                        // d = 128 kernel, the mean square of every row of X
  // float16 operands of the forward GEMMs (see k_encode_rows_f16): the encoded X [N][d], the factor the epilogues
  // multiply each accumulator row by [N], and R^T as float16 [d][d]
  size_t x16, rowacc, rt16;
  bool f16;             // those three exist
  size_t total;
  long long ldt;
  int P, bn, loss_blocks, norm_n;
};

// The token GEMMs of the forward pass take float16 operands whenever R would otherwise enter as a single bf16 term
// (d > 512 by default), unless the configuration asks for bf16.
static bool forward_is_f16(const kt_config* cfg, int64_t d, int gather_batch) {
  (void)gather_batch;
  const int terms = cfg == nullptr ? 0 : cfg->forward_terms;
  const bool one_term = terms == 1 || (terms != 2 && d > 512);
  return one_term && (cfg == nullptr || cfg->forward_bf16 == 0);
}

// cfg == null: the default configuration (no momentum buffer, no RMSNorm factors).
// gather_batch > 0: the layout of kt_fit_shared (N = batch * rows per sample): the dense bf16 matrix is the gathered
// minibatch, and the sample ids of kIdsChunk steps and the buffers' base pointers live in the workspace too.
static WsLayout make_layout(int64_t N, int64_t d, int32_t x_dtype, const kt_config* cfg,
                            int gather_batch = 0) {
  const bool adam = cfg != nullptr && cfg->optimizer == 1;
  // (d = 128: the single-pass kernel reads its own float16 encoding of X, whatever X's type)
  const bool xcopy = x_dtype == KT_F32 || gather_batch > 0 ||
                     (d == kFsD && (cfg == nullptr || (cfg->small_d_fused != 0 && cfg->loss_mode == 0)));
  // Y kept for the backward pass, unless the backward recomputes it or the single-pass kernel (d = 128, per-token
  // loss) does forward and backward together
  const bool single_pass = d == kFsD && (cfg == nullptr || (cfg->small_d_fused != 0 && cfg->loss_mode == 0));
  const bool keep_y = (cfg == nullptr || cfg->backward_mode != 1) && !single_pass;
  const bool y_f32 = cfg != nullptr && cfg->backward_mode == 2;
  WsLayout L;
  memset(&L, 0, sizeof(L));
  L.bn = (d % 256 == 0) ? 128 : 64;  // columns per moment record: half a GEMM column tile
  L.P = static_cast<int>(d / L.bn);
  L.ldt = static_cast<long long>(align_up(static_cast<size_t>(N), 64));
  L.loss_blocks = static_cast<int>((N + 255) / 256);
  L.norm_n = static_cast<int>((d / 32) * (d / 32));
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t dd = static_cast<size_t>(d) * d;
  L.rt_hi = take(dd * 2);
  L.rt_lo = take(dd * 2);
  L.r_hi = take(dd * 2);
  L.r_lo = take(dd * 2);
  L.z_hi = take(dd * 2);
  L.z_lo = take(dd * 2);
  L.w_hi = take(dd * 2);
  L.w_lo = take(dd * 2);
  L.fbuf = take(dd * 4);
  L.dr = take(dd * 4);
  L.xb = take(xcopy ? static_cast<size_t>(N) * d * 2 : 0);
  L.xt = take(static_cast<size_t>(d) * L.ldt * 2);
  L.gt = take(static_cast<size_t>(d) * L.ldt * 2);
  L.ybuf = take(keep_y ? static_cast<size_t>(N) * d * (y_f32 ? 4 : 2) : 0);
  L.yexp = take((keep_y && !y_f32) ? static_cast<size_t>(L.P) * N : 0);
  L.partial = take(static_cast<size_t>(L.P) * N * 16);
  L.coef = take(static_cast<size_t>(N) * 16);
  L.moments = take(static_cast<size_t>(N) * 16);
  // at least 256 entries: the fused d = 128 kernel writes one partial per CTA here
  L.block_loss = take(static_cast<size_t>(L.loss_blocks > 256 ? L.loss_blocks : 256) * 8);
  L.block_deg = take(static_cast<size_t>(L.loss_blocks > 256 ? L.loss_blocks : 256) * 4);
  L.norm_blocks = take(static_cast<size_t>(L.norm_n > 1024 ? L.norm_n : 1024) * 8);
  L.rowmax = take(static_cast<size_t>(N) * 4);
  L.rowmin = take(static_cast<size_t>(N) * 4);
  L.qerr = take(static_cast<size_t>(L.P) * N * 4);
  L.colpart = take(static_cast<size_t>(d / 32) * d * 4);
  L.diag = take(static_cast<size_t>(d) * 4);
  L.pvec = take(static_cast<size_t>(d) * 4 * 2);
  {
    const SplitPlan sp = plan_split_k(d, N);
    int parts = sp.splits > 1 ? sp.splits : 0;
    if (d == kFsD && parts < 256) parts = 256;  // per-CTA partial dR of the fused d = 128 kernel
    L.splitk = take(static_cast<size_t>(parts) * dd * 4);
  }
  L.small = take(d <= 512 ? 6 * dd * 4 + 4096 : 0);
  L.adam_m = take(adam ? dd * 4 : 0);
  L.gather_ids = take(gather_batch > 0 ? static_cast<size_t>(kIdsChunk) * gather_batch * 4 : 0);
  L.gather_bases = take(gather_batch > 0 ? static_cast<size_t>(kMaxSharedBufs) * 8 : 0);
  L.flat = take(static_cast<size_t>(L.loss_blocks) * 8 * 3 + 64);
  // (d = 128: the single-pass kernel's per-row mean square of X lives here too)
  L.rowscale = take(((cfg != nullptr && cfg->rmsnorm != 0) || d == kFsD) ? static_cast<size_t>(N) * 4 : 0);
  const bool f16 = forward_is_f16(cfg, d, gather_batch);
  L.f16 = f16;
  L.x16 = take(f16 ? static_cast<size_t>(N) * d * 2 : 0);
  L.rowacc = take(f16 ? static_cast<size_t>(N) * 4 : 0);
  L.rt16 = take(f16 ? dd * 2 : 0);
  L.total = off;
  return L;
}

}  // namespace kt

struct kt_ctx {
  kt_config cfg;
  cudaStream_t stream;
  int device;
  int sm_count;
  uint8_t* ws;
  size_t ws_bytes;
  kt::DeviceBlock* d_blk;
  kt::DeviceBlock* h_blk;  // pinned
  kt::EncodeTiledFn encode;
  // profiling (kt_profile_begin/kt_profile_end)
  long long launches;       // kernels launched since kt_profile_begin
  bool prof_on;
  cudaEvent_t* prof_ev;     // 2 * kProfPairs events, created on first use
  int prof_used;            // pairs recorded
  unsigned char* prof_cat;  // category of each pair
  // kt_fit_sharded: the caller's sum over shards, called on the host while the step is being enqueued
  kt_reduce_fn reduce_fn;
  void* reduce_user;
  double rows_total;        // tokens of all shards (0 outside kt_fit_sharded: the rows of the call's own X)
};

namespace kt {

#define KT_CUDA(call)                       \
  do {                                      \
    if ((call) != cudaSuccess) {            \
      (void)cudaGetLastError();             \
      return KT_ERR_CUDA;                   \
    }                                       \
  } while (0)
#define KT_LAUNCH_CHECK()          \
  do {                             \
    KT_CUDA(cudaGetLastError());   \
    ++ctx->launches;               \
  } while (0)
#define KT_TRY(expr)                 \
  do {                               \
    kt_status st__ = (expr);         \
    if (st__ != KT_OK) return st__;  \
  } while (0)

static bool use_fused(const kt_ctx* ctx, int d);
// bound of every device-side wait of the launches of this context (kt_config.wait_limit_ms)
static unsigned long long wait_limit_ns(const kt_ctx* ctx) {
  return ctx->cfg.wait_limit_ms > 0 ? static_cast<unsigned long long>(ctx->cfg.wait_limit_ms) * 1000000ull
                                    : kDefaultWaitLimitNs;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static kt_status check_x(const kt_mat& X, int64_t* N, int64_t* d) {
  if (X.data == nullptr) return KT_ERR_INVALID_ARG;
  if (X.dtype != KT_BF16 && X.dtype != KT_F32) return KT_ERR_INVALID_ARG;
  if (X.rows < 1 || X.cols < 128 || X.cols % 128 != 0 || X.ld < X.cols) return KT_ERR_SHAPE;
  if (X.rows > 0x7fffff00ll || X.cols > 65536) return KT_ERR_SHAPE;
  const int64_t es = (X.dtype == KT_BF16) ? 2 : 4;
  if (!aligned16(X.data) || (X.ld * es) % 16 != 0) return KT_ERR_ALIGN;
  *N = X.rows;
  *d = X.cols;
  return KT_OK;
}

static kt_status check_ws(const kt_ctx* ctx, const WsLayout& L) {
  if (ctx->ws == nullptr || ctx->ws_bytes < L.total) return KT_ERR_WORKSPACE;
  return KT_OK;
}

// Sum over the shards of a sharded fit (no-op otherwise): hands the device buffer to the caller's hook, which
// enqueues an in-place sum all-reduce on the context's stream.
static kt_status reduce_shards(kt_ctx* ctx, void* dev_ptr, int64_t count, kt_dtype dtype) {
  if (ctx->reduce_fn == nullptr) return KT_OK;
  return ctx->reduce_fn(ctx->reduce_user, dev_ptr, count, static_cast<int32_t>(dtype), ctx->stream) == 0
             ? KT_OK
             : KT_ERR_REDUCE;
}
static double mean_rows(const kt_ctx* ctx, int N) { return ctx->rows_total > 0.0 ? ctx->rows_total : N; }

// bf16 matrix of `rows` rows, `k_extent` valid elements per row, leading
// dimension ld (elements); tiles of box_rows x 64 elements, 128-byte swizzle,
// out-of-range elements read as zero.
static kt_status make_tmap(const kt_ctx* ctx, CUtensorMap* tm, const void* base, uint64_t k_extent, uint64_t rows,
                           uint64_t ld, uint32_t box_rows) {
  cuuint64_t dims[2] = {k_extent, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK), box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = ctx->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? KT_OK : KT_ERR_CUDA;
}

// Per-device, per-kernel set-up done once (the opt-in to large dynamic shared memory, and for kernels launched as
// clusters the number of clusters the device can hold at once).  Guarded by a mutex: contexts may live on several
// host threads.  Devices beyond the table are set up on every launch.
constexpr int kMaxDevices = 64;
struct KernelSetup {
  bool done[kMaxDevices];
  int slots[kMaxDevices];
};
static std::mutex g_setup_mutex;

template <int BN, int EPI, int CTAS>
static kt_status gemm_setup(kt_ctx* ctx, int* slots_out) {
  static KernelSetup ks = {};
  const int smem = GemmSmem<BN, CTAS>::kTotal;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  const bool cached = ctx->device >= 0 && ctx->device < kMaxDevices;
  if (cached && ks.done[ctx->device]) {
    *slots_out = ks.slots[ctx->device];
    return KT_OK;
  }
  KT_CUDA(cudaFuncSetAttribute(gemm_tn_kernel<BN, EPI, CTAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  int slots = ctx->sm_count / CTAS;
  if (CTAS > 1) {
    // a persistent kernel wants every cluster resident at once: ask how many the device can co-schedule (an SM
    // that cannot pair up inside its GPC holds none) instead of assuming sm_count / CTAS
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(static_cast<unsigned>(slots * CTAS));
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = CTAS;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tn_kernel<BN, EPI, CTAS>, &cfg) == cudaSuccess && n > 0) {
      if (n < slots) slots = n;
    } else {
      (void)cudaGetLastError();
    }
  }
  if (cached) {
    ks.done[ctx->device] = true;
    ks.slots[ctx->device] = slots;
  }
  *slots_out = slots;
  return KT_OK;
}

template <int BN, int EPI, int CTAS>
static kt_status launch_gemm_inst(kt_ctx* ctx, const GemmParams& p, int cat) {
  const int smem = GemmSmem<BN, CTAS>::kTotal;
  int slots = 0;
  KT_TRY((gemm_setup<BN, EPI, CTAS>(ctx, &slots)));
  // one CTA (or one pair of CTAs) per work unit, at most one CTA per SM and no more than fit at once
  const int units = p.m_tiles * p.n_tiles * p.k_splits;
  const int grid = (units < slots ? units : slots) * CTAS;
  const bool rec = ctx->prof_on && ctx->prof_used < kProfPairs;
  if (rec) KT_CUDA(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used], ctx->stream));
  if (CTAS == 1) {
    gemm_tn_kernel<BN, EPI, CTAS><<<grid, kGemmThreads, smem, ctx->stream>>>(p);
  } else {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kGemmThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = ctx->stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = CTAS;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    KT_CUDA(cudaLaunchKernelEx(&cfg, gemm_tn_kernel<BN, EPI, CTAS>, p));
  }
  KT_LAUNCH_CHECK();
  if (rec) {
    KT_CUDA(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used + 1], ctx->stream));
    ctx->prof_cat[ctx->prof_used++] = static_cast<unsigned char>(cat);
  }
  return KT_OK;
}

struct Operand {
  const void* base;
  uint64_t ld;
};

// D (M x N) = sum_q A_q (M x K) * B_q (N x K)^T with the epilogue EPI.
template <int EPI>
static kt_status run_gemm(kt_ctx* ctx, int M, int N, int K, int terms, const Operand* A, const Operand* B,
                          GemmParams& p, int cat) {
  const int bn = (N % 256 == 0) ? 256 : 128;
  // 256-wide tiles with more than one row tile run on pairs of CTAs (256 x 256 tiles, each CTA loading half of B)
  const int ctas = (bn == 256 && M > kBM && ctx->cfg.cta_pairs != 0 && ctx->sm_count % 2 == 0) ? 2 : 1;
  p.terms = terms;
  p.M = M;
  p.N = N;
  p.K = K;
  p.m_tiles = (M + kBM * ctas - 1) / (kBM * ctas);
  p.n_tiles = N / bn;
  if (p.k_splits < 1) {
    p.k_splits = 1;
    p.kb_per_split = (K + kBK - 1) / kBK;
  }
  p.err_word = &ctx->d_blk->sc.err_word;
  p.wait_limit_ns = wait_limit_ns(ctx);
  // 32-byte stores need every row start on a 32-byte boundary (the column offsets are multiples of 32 floats)
  p.out_sector_aligned = (p.out != nullptr && (reinterpret_cast<uintptr_t>(p.out) & 31u) == 0 && (p.ldo & 7) == 0 &&
                          (p.split_stride & 7) == 0)
                             ? 1
                             : 0;
  for (int q = 0; q < terms; ++q) {
    KT_TRY(make_tmap(ctx, &p.tmA[q], A[q].base, K, M, A[q].ld, kBM));
    KT_TRY(make_tmap(ctx, &p.tmB[q], B[q].base, K, N, B[q].ld, bn / ctas));
  }
  if (ctas == 2) return launch_gemm_inst<256, EPI, 2>(ctx, p, cat);
  if (bn == 256) return launch_gemm_inst<256, EPI, 1>(ctx, p, cat);
  return launch_gemm_inst<128, EPI, 1>(ctx, p, cat);
}

static GemmParams blank_params() {
  GemmParams p;
  memset(&p, 0, sizeof(p));
  return p;
}

template <typename T>
static T* at(kt_ctx* ctx, size_t off) {
  return reinterpret_cast<T*>(ctx->ws + off);
}

// ---------------------------------------------------------------- X ingest
struct XView {
  const __nv_bfloat16* xb;  // bf16 rows
  long long ldx;
  const float* row_scale;   // RMSNorm factor of every row (kt_config.rmsnorm), or null
  const float* row_ms;      // single-pass d = 128 kernel: mean square of every row of X
  const __half* x16;        // the rows in the float16 encoding of the forward GEMMs (dense, N x d), or null
  const float* acc_scale;   // what the forward GEMMs' epilogues multiply each accumulator row by, or null: the
                            // RMSNorm factor, times the inverse of the float16 encoding's row factor
};

// Completes a view whose bf16 rows (and RMSNorm factors) are set: the float16 encoding when this problem uses it.
static kt_status finish_view(kt_ctx* ctx, int64_t N, int64_t d, const WsLayout& L, XView* v);

// The single-pass d = 128 kernel's own encoding of X (row-normalised float16, see k_encode_rows_128) and each encoded
// row's mean square: one pass over X, needed once per X.
static kt_status fused_encode(kt_ctx* ctx, const kt_mat& X, const WsLayout& L, XView* v);

// RMSNorm mode: the factor 1/sqrt(mean(x^2) + eps) of every row, applied later to the float32 accumulator rows of
// X R (an orthogonal R keeps the norm of a row); a float32 X is rounded to its bf16 copy in the same pass.
static kt_status row_scale_x(kt_ctx* ctx, const kt_mat& X, const WsLayout& L, XView* v) {
  const int d = static_cast<int>(X.cols);
  float* rsc = at<float>(ctx, L.rowscale);
  const unsigned rows = static_cast<unsigned>(X.rows);
  if (X.dtype == KT_BF16) {
    k_row_scale<__nv_bfloat16><<<rows, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(X.data), X.ld, d,
                                                              ctx->cfg.rms_eps, rsc, nullptr, nullptr, 0, 0, nullptr);
    v->xb = static_cast<const __nv_bfloat16*>(X.data);
    v->ldx = X.ld;
  } else {
    __nv_bfloat16* xb = at<__nv_bfloat16>(ctx, L.xb);
    k_row_scale<float><<<rows, 256, 0, ctx->stream>>>(static_cast<const float*>(X.data), X.ld, d, ctx->cfg.rms_eps,
                                                      rsc, xb, nullptr, 0, 0, nullptr);
    v->xb = xb;
    v->ldx = d;
  }
  KT_LAUNCH_CHECK();
  v->row_scale = rsc;
  return KT_OK;
}

// forward-only view: bf16 X is used in place, float32 X is rounded into the workspace
// want_scale = false: no RMSNorm factors even when kt_config.rmsnorm is on (the single-pass d = 128 kernel: the
// per-token kurtosis, and with it its gradient with respect to X R, does not depend on the scale of a row).
static kt_status ingest_x_forward(kt_ctx* ctx, const kt_mat& X, const WsLayout& L, XView* v, bool want_scale = true) {
  const int64_t N = X.rows, d = X.cols;
  v->row_scale = nullptr;
  v->row_ms = nullptr;
  if (ctx->cfg.rmsnorm != 0 && want_scale) {
    KT_TRY(row_scale_x(ctx, X, L, v));
    return finish_view(ctx, N, d, L, v);
  }
  if (X.dtype == KT_BF16) {
    v->xb = static_cast<const __nv_bfloat16*>(X.data);
    v->ldx = X.ld;
    return finish_view(ctx, N, d, L, v);
  }
  __nv_bfloat16* xb = at<__nv_bfloat16>(ctx, L.xb);
  const long long pairs = N * d / 2;
  k_cast_x<<<static_cast<unsigned>((pairs + 255) / 256), 256, 0, ctx->stream>>>(static_cast<const float*>(X.data),
                                                                                X.ld, N, static_cast<int>(d), xb);
  KT_LAUNCH_CHECK();
  v->xb = xb;
  v->ldx = d;
  return finish_view(ctx, N, d, L, v);
}

// X^T of a bf16 X (no dense copy needed): the wide-load transpose.
static kt_status transpose_x_bf16(kt_ctx* ctx, const __nv_bfloat16* X, long long ld, int N, int d, const WsLayout& L) {
  dim3 grid(d / 128, (N + 63) / 64);
  k_transpose_x_bf16<<<grid, 256, 0, ctx->stream>>>(X, ld, N, d, at<__nv_bfloat16>(ctx, L.xt), L.ldt);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

// view for loss + gradient: also builds X^T (the token dimension becomes contiguous)
static kt_status ingest_x_full(kt_ctx* ctx, const kt_mat& X, const WsLayout& L, XView* v) {
  const int N = static_cast<int>(X.rows), d = static_cast<int>(X.cols);
  dim3 grid(d / 64, (N + 63) / 64), block(32, 8);
  __nv_bfloat16* xt = at<__nv_bfloat16>(ctx, L.xt);
  v->row_scale = nullptr;
  v->row_ms = nullptr;
  if (ctx->cfg.rmsnorm != 0) {
    KT_TRY(row_scale_x(ctx, X, L, v));
    KT_TRY(transpose_x_bf16(ctx, v->xb, v->ldx, N, d, L));
  } else if (X.dtype == KT_BF16) {
    KT_TRY(transpose_x_bf16(ctx, static_cast<const __nv_bfloat16*>(X.data), X.ld, N, d, L));
    v->xb = static_cast<const __nv_bfloat16*>(X.data);
    v->ldx = X.ld;
  } else {
    __nv_bfloat16* xb = at<__nv_bfloat16>(ctx, L.xb);
    k_prepare_x<float><<<grid, block, 0, ctx->stream>>>(static_cast<const float*>(X.data), X.ld, N, d, xt, L.ldt, xb);
    KT_LAUNCH_CHECK();
    v->xb = xb;
    v->ldx = d;
  }
  return finish_view(ctx, N, d, L, v);
}

static kt_status finish_view(kt_ctx* ctx, int64_t N, int64_t d, const WsLayout& L, XView* v) {
  v->x16 = nullptr;
  v->acc_scale = v->row_scale;
  if (!L.f16) return KT_OK;
  __half* x16 = at<__half>(ctx, L.x16);
  float* acc = at<float>(ctx, L.rowacc);
  k_encode_rows_f16<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(v->xb, v->ldx, static_cast<int>(d), x16,
                                                                       v->row_scale, acc);
  KT_LAUNCH_CHECK();
  v->x16 = x16;
  v->acc_scale = acc;
  return KT_OK;
}

// ------------------------------------------------------------ forward pieces
// How many bf16 terms of R the token GEMMs use: 1 (R rounded to bf16) or 2 (hi + lo, ~16 significant bits).
// Automatic choice: 2 for d <= 512.  With few channels the rounding of R does not average out: every token whose
// energy sits in the same few channels sees the same rounded rows of R, and one bf16 term then misses the 1e-3
// loss tolerance (measured 2.2e-3 on single-head KV data with two outlier channels at d = 128).
static int forward_terms(const kt_ctx* ctx, int d, long long N) {
  (void)N;
  const int t = ctx->cfg.forward_terms;
  if (t == 1 || t == 2) return t;
  return d <= 512 ? 2 : 1;
}

// R^T as float16 for the forward GEMMs of a problem that uses the float16 encoding.  Inside a fit the orthogonal
// step keeps it up to date together with the bf16 forms (k_series_term, k_polish_apply).
static kt_status cast_rt16(kt_ctx* ctx, const float* R, int d, const WsLayout& L) {
  if (!L.f16) return KT_OK;
  dim3 grid(d / 32, d / 32), block(32, 8);
  k_rt_f16<<<grid, block, 0, ctx->stream>>>(R, d, at<__half>(ctx, L.rt16));
  KT_LAUNCH_CHECK();
  return KT_OK;
}

static kt_status cast_rt(kt_ctx* ctx, const float* R, int d, long long N, const WsLayout& L) {
  dim3 grid(d / 32, d / 32), block(32, 8);
  k_split_bf16<true><<<grid, block, 0, ctx->stream>>>(
      R, d, at<__nv_bfloat16>(ctx, L.rt_hi), forward_terms(ctx, d, N) == 2 ? at<__nv_bfloat16>(ctx, L.rt_lo) : nullptr,
      d);
  KT_LAUNCH_CHECK();
  KT_TRY(cast_rt16(ctx, R, d, L));
  return KT_OK;
}

// Operands of Y = X R for the token GEMMs: X against R^T hi (and lo) in bf16, or the float16 encoding of X against
// R^T as float16.  fwd_operands() also sets the parameters that go with the choice (operand type, row factors).
struct FwdOperands {
  Operand A[2], B[2];
  int terms;
};
static FwdOperands fwd_operands(kt_ctx* ctx, const XView& xv, int d, long long N, const WsLayout& L, GemmParams* p) {
  FwdOperands f;
  p->row_scale = xv.acc_scale;
  if (xv.x16 != nullptr) {
    f.terms = 1;
    f.A[0] = f.A[1] = Operand{xv.x16, static_cast<uint64_t>(d)};
    f.B[0] = f.B[1] = Operand{at<__half>(ctx, L.rt16), static_cast<uint64_t>(d)};
    p->f16_operands = 1;
    return f;
  }
  f.terms = forward_terms(ctx, d, N);
  f.A[0] = f.A[1] = Operand{xv.xb, static_cast<uint64_t>(xv.ldx)};
  f.B[0] = Operand{at<__nv_bfloat16>(ctx, L.rt_hi), static_cast<uint64_t>(d)};
  f.B[1] = Operand{at<__nv_bfloat16>(ctx, L.rt_lo), static_cast<uint64_t>(d)};
  return f;
}

static bool y_stored_f32(const kt_ctx* ctx) { return ctx->cfg.backward_mode == 2; }

// moments + loss for the rows of xv; R^T must already be in rt_hi.
// keep_y: the epilogue also stores the Y tile into the workspace (for the backward pass), as float32 or float16.
// err_to_nan: *hist_slot receives NaN when a device-side wait of this call ran out (for callers that never read
// the status word on the host).
static kt_status forward_loss(kt_ctx* ctx, const XView& xv, int N, int d, const WsLayout& L, double* hist_slot,
                              bool keep_y = false, bool err_to_nan = false) {
  GemmParams p = blank_params();
  p.partial = at<float4>(ctx, L.partial);
  if (keep_y && y_stored_f32(ctx)) {
    p.out = at<float>(ctx, L.ybuf);
    p.ldo = d;
  } else if (keep_y) {
    p.out16 = at<__half>(ctx, L.ybuf);
    p.out16_exp = at<unsigned char>(ctx, L.yexp);
    p.ldo = d;
  }
  const double n_mean = mean_rows(ctx, N);
  const FwdOperands f = fwd_operands(ctx, xv, d, N, L, &p);
  KT_TRY(run_gemm<kMoments>(ctx, N, d, d, f.terms, f.A, f.B, p, kCatForward));
  k_moments_finalize<<<L.loss_blocks, 256, 0, ctx->stream>>>(at<float4>(ctx, L.partial), L.P, N, d, L.bn,
                                                            ctx->cfg.kappa_target, at<float4>(ctx, L.moments),
                                                            at<float4>(ctx, L.coef), at<double>(ctx, L.block_loss),
                                                            at<unsigned int>(ctx, L.block_deg), n_mean,
                                                            xv.row_scale);
  KT_LAUNCH_CHECK();
  if (ctx->cfg.loss_mode == 1) {
    // one kurtosis over all N d entries: merge the rows' moments, then hand every row the layer's coefficients
    const int nb = L.loss_blocks;
    // L.flat is 256-byte aligned: the float4 of global coefficients first (16-byte aligned), the mean at +16,
    // three doubles for a sharded fit's central sums at +24, the three per-block arrays from +64
    float4* cg = at<float4>(ctx, L.flat);
    double* mean = at<double>(ctx, L.flat + 16);
    double* b2 = at<double>(ctx, L.flat + 64);
    double* b3 = b2 + nb;
    double* b4 = b3 + nb;
    k_flat_mean<<<nb, 256, 0, ctx->stream>>>(at<float4>(ctx, L.moments), N, at<double>(ctx, L.block_loss));
    KT_LAUNCH_CHECK();
    k_final_sum<<<1, 256, 0, ctx->stream>>>(at<double>(ctx, L.block_loss), nb, 1.0 / n_mean, mean, nullptr, nullptr,
                                            nullptr);
    KT_LAUNCH_CHECK();
    KT_TRY(reduce_shards(ctx, mean, 1, KT_F64));  // the mean of the whole batch
    k_flat_central<<<nb, 256, 0, ctx->stream>>>(at<float4>(ctx, L.moments), N, mean, b2, b3, b4);
    KT_LAUNCH_CHECK();
    const long long n_all = static_cast<long long>(n_mean);
    if (ctx->reduce_fn != nullptr) {
      // sharded: this shard's three central sums (in the doubles after the mean), summed over the shards
      double* s3 = at<double>(ctx, L.flat + 24);
      const double* blocks[3] = {b2, b3, b4};
      for (int i = 0; i < 3; ++i) {
        k_final_sum<<<1, 256, 0, ctx->stream>>>(blocks[i], nb, 1.0, s3 + i, nullptr, nullptr, nullptr);
        KT_LAUNCH_CHECK();
      }
      KT_TRY(reduce_shards(ctx, s3, 3, KT_F64));
      k_flat_finalize<<<1, 256, 0, ctx->stream>>>(s3, s3 + 1, s3 + 2, 1, n_all, d, ctx->cfg.kappa_target, mean,
                                                  &ctx->d_blk->sc, hist_slot, cg);
    } else {
      k_flat_finalize<<<1, 256, 0, ctx->stream>>>(b2, b3, b4, nb, n_all, d, ctx->cfg.kappa_target, mean,
                                                  &ctx->d_blk->sc, hist_slot, cg);
    }
    KT_LAUNCH_CHECK();
    k_flat_fill<<<nb, 256, 0, ctx->stream>>>(cg, N, at<float4>(ctx, L.coef), xv.row_scale);
    KT_LAUNCH_CHECK();
    return KT_OK;
  }
  k_final_sum<<<1, 256, 0, ctx->stream>>>(at<double>(ctx, L.block_loss), L.loss_blocks, 1.0 / n_mean,
                                          &ctx->d_blk->sc.loss, hist_slot, at<unsigned int>(ctx, L.block_deg),
                                          &ctx->d_blk->sc.deg_rows, err_to_nan ? &ctx->d_blk->sc.err_word : nullptr);
  KT_LAUNCH_CHECK();
  if (hist_slot != nullptr) KT_TRY(reduce_shards(ctx, hist_slot, 1, KT_F64));  // the loss of the whole batch
  return KT_OK;
}

// dR = X^T G with G from the saved row coefficients and Y: either the Y tile is recomputed by a second pass of the
// forward GEMM (nothing of Y ever reaches memory), or the Y the forward pass kept is read back by an element-wise
// kernel.  A float32 Y (backward_mode 2) gives the recomputing pass's bits: the same float32 expression on the same
// accumulator values.  The float16 Y (the default) is those values rounded to 11 significant bits.
static bool keep_y_for_backward(const kt_ctx* ctx) { return ctx->cfg.backward_mode != 1; }

// dr_hi != null: the split-K sum also leaves bf16(dR) there (only when the sum runs; see dr_hi_from_backward()).
static kt_status backward(kt_ctx* ctx, const XView& xv, int N, int d, const WsLayout& L, float* dR,
                          __nv_bfloat16* dr_hi = nullptr) {
  if (keep_y_for_backward(ctx) && y_stored_f32(ctx)) {
    dim3 grid((N + 63) / 64, d / 64);
    k_grad_from_y<<<grid, 256, 0, ctx->stream>>>(at<float>(ctx, L.ybuf), at<float4>(ctx, L.coef), N, d,
                                                 at<__nv_bfloat16>(ctx, L.gt), L.ldt);
    KT_LAUNCH_CHECK();
  } else if (keep_y_for_backward(ctx)) {
    dim3 grid((N + 127) / 128, d / 64);
    k_grad_from_y16<<<grid, 256, 0, ctx->stream>>>(at<__half>(ctx, L.ybuf), at<unsigned char>(ctx, L.yexp), L.bn,
                                                   at<float4>(ctx, L.coef), N, d, at<__nv_bfloat16>(ctx, L.gt),
                                                   L.ldt);
    KT_LAUNCH_CHECK();
  } else {
    GemmParams p = blank_params();
    p.coef = at<float4>(ctx, L.coef);
    p.gt = at<__nv_bfloat16>(ctx, L.gt);
    p.ldg = L.ldt;
    const FwdOperands f = fwd_operands(ctx, xv, d, N, L, &p);
    KT_TRY(run_gemm<kGrad>(ctx, N, d, d, f.terms, f.A, f.B, p, kCatBackwardA));
  }
  GemmParams p2 = blank_params();
  const SplitPlan sp = plan_split_k(d, N);
  p2.out = sp.splits > 1 ? at<float>(ctx, L.splitk) : dR;
  p2.ldo = d;
  p2.k_splits = sp.splits;
  p2.kb_per_split = sp.kb_per_split;
  p2.split_stride = static_cast<long long>(d) * d;
  Operand A2{at<__nv_bfloat16>(ctx, L.xt), static_cast<uint64_t>(L.ldt)},
      B2{at<__nv_bfloat16>(ctx, L.gt), static_cast<uint64_t>(L.ldt)};
  KT_TRY(run_gemm<kStoreF32>(ctx, d, d, N, 1, &A2, &B2, p2, kCatBackwardB));
  if (sp.splits > 1) {
    const long long n = static_cast<long long>(d) * d;
    k_sum_splits<<<static_cast<unsigned>((n / 4 + 255) / 256), 256, 0, ctx->stream>>>(at<float>(ctx, L.splitk),
                                                                                       sp.splits, n, n, dR, dr_hi);
    KT_LAUNCH_CHECK();
  }
  return KT_OK;
}

static bool use_small_orth(const kt_ctx* ctx, int d);

static kt_status loss_grad_async(kt_ctx* ctx, const XView& xv, int N, int d, const WsLayout& L, const float* R,
                                 float* dR, double* hist_slot, bool rt_current, __nv_bfloat16* dr_hi = nullptr) {
  if (!rt_current) KT_TRY(cast_rt(ctx, R, d, N, L));
  else if (use_small_orth(ctx, d)) KT_TRY(cast_rt16(ctx, R, d, L));  // (the one-launch step leaves the bf16 forms only)
  KT_TRY(forward_loss(ctx, xv, N, d, L, hist_slot, keep_y_for_backward(ctx)));
  KT_TRY(backward(ctx, xv, N, d, L, dR, dr_hi));
  KT_TRY(reduce_shards(ctx, dR, static_cast<int64_t>(d) * d, KT_F32));  // the gradient of the whole batch
  return KT_OK;
}

// d = 128: loss and gradient in one pass over X (fused_small_kernel), then fixed-order sums over the CTAs.
// (the single-pass kernel needs each row's coefficients before the row leaves the SM: per-token loss only)
static bool use_fused(const kt_ctx* ctx, int d) {
  return d == kFsD && ctx->cfg.small_d_fused != 0 && ctx->cfg.loss_mode == 0;
}

static kt_status fused_encode(kt_ctx* ctx, const kt_mat& X, const WsLayout& L, XView* v) {
  const int N = static_cast<int>(X.rows);
  float* ms = at<float>(ctx, L.rowscale);
  __half* x16 = at<__half>(ctx, L.xb);
  const unsigned grid = static_cast<unsigned>((N + 15) / 16);
  if (X.dtype == KT_BF16)
    k_encode_rows_128<__nv_bfloat16><<<grid, 256, 0, ctx->stream>>>(static_cast<const __nv_bfloat16*>(X.data), X.ld, N,
                                                                    x16, ms, nullptr, 0, 0, nullptr);
  else
    k_encode_rows_128<float><<<grid, 256, 0, ctx->stream>>>(static_cast<const float*>(X.data), X.ld, N, x16, ms,
                                                            nullptr, 0, 0, nullptr);
  KT_LAUNCH_CHECK();
  v->xb = reinterpret_cast<const __nv_bfloat16*>(x16);   // 16-bit words: float16 here
  v->ldx = kFsD;
  v->row_scale = nullptr;
  v->row_ms = ms;
  return KT_OK;
}

// The single-pass kernel alone: leaves per-CTA partials of dR, of the loss and of the skipped-row count in the
// workspace, described by *fp (to be summed by k_fused_finish or by the first phase of small_orth_kernel).
static kt_status fused_launch(kt_ctx* ctx, const XView& xv, int N, const WsLayout& L, const float* R,
                              double* hist_slot, bool rt_current, FusedPartials* fp) {
  const int d = kFsD;
  if (!rt_current) {
    // the kernel's second operand is Rc^T, R with every row's mean taken off (see first_order_term)
    k_center_split_128<<<kFsD, 128, 0, ctx->stream>>>(R, at<__nv_bfloat16>(ctx, L.rt_hi),
                                                      at<__nv_bfloat16>(ctx, L.rt_lo));
    KT_LAUNCH_CHECK();
  }
  {
    static bool attr_done[kMaxDevices] = {false};
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    const bool cached = ctx->device >= 0 && ctx->device < kMaxDevices;
    if (!cached || !attr_done[ctx->device]) {
      KT_CUDA(cudaFuncSetAttribute(fused_small_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   FusedCfg<1>::kSmem));
      KT_CUDA(cudaFuncSetAttribute(fused_small_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   FusedCfg<2>::kSmem));
      if (cached) attr_done[ctx->device] = true;
    }
  }
  FusedParams p;
  memset(&p, 0, sizeof(p));
  // R enters the single-pass kernel as one bf16 term unless two are asked for explicitly: the loss, whose error
  // under a rounded R is systematic at this size (see forward_terms()), is corrected to first order from the
  // gradient the same pass yields (first_order_term), which costs nothing next to a second term's MMAs
  const int terms = ctx->cfg.forward_terms == 2 ? 2 : 1;
  const bool correct_loss = ctx->cfg.forward_terms == 0;
  p.N = N;
  p.n_mean = mean_rows(ctx, N);
  p.tiles = (N + 127) / 128;
  p.kappa_t = ctx->cfg.kappa_target;
  p.wait_limit_ns = wait_limit_ns(ctx);
  p.dr_partial = at<float>(ctx, L.splitk);
  p.loss_partial = at<double>(ctx, L.block_loss);
  p.deg_partial = at<unsigned int>(ctx, L.block_deg);
  p.err_word = &ctx->d_blk->sc.err_word;
  p.row_ms = xv.row_ms;
  KT_TRY(make_tmap(ctx, &p.tmX, xv.xb, d, N, xv.ldx, 128));
  KT_TRY(make_tmap(ctx, &p.tmRhi, at<__nv_bfloat16>(ctx, L.rt_hi), d, d, d, 128));
  KT_TRY(make_tmap(ctx, &p.tmRlo, at<__nv_bfloat16>(ctx, L.rt_lo), d, d, d, 128));
  int grid = p.tiles < ctx->sm_count ? p.tiles : ctx->sm_count;
  if (grid > 256) grid = 256;
  const bool rec = ctx->prof_on && ctx->prof_used < kProfPairs;
  if (rec) KT_CUDA(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used], ctx->stream));
  if (terms == 2)
    fused_small_kernel<2><<<grid, kFsThreads, FusedCfg<2>::kSmem, ctx->stream>>>(p);
  else
    fused_small_kernel<1><<<grid, kFsThreads, FusedCfg<1>::kSmem, ctx->stream>>>(p);
  KT_LAUNCH_CHECK();
  if (rec) {
    KT_CUDA(cudaEventRecord(ctx->prof_ev[2 * ctx->prof_used + 1], ctx->stream));
    ctx->prof_cat[ctx->prof_used++] = static_cast<unsigned char>(kCatFused);
  }
  fp->dr_part = p.dr_partial;
  fp->parts = grid;
  fp->loss_part = p.loss_partial;
  fp->deg_part = p.deg_partial;
  fp->loss_scale = 1.0 / p.n_mean;
  fp->dr_scale = static_cast<float>(4.0 / (p.n_mean * 128.0));
  fp->correct = correct_loss ? 1 : 0;
  fp->rowdot = at<double>(ctx, L.norm_blocks);
  fp->hist_slot = hist_slot;
  return KT_OK;
}

// d = 128: loss and gradient in one pass over X, then the fixed-order sums over the CTAs' partials.
static kt_status fused_loss_grad_async(kt_ctx* ctx, const XView& xv, int N, const WsLayout& L, const float* R,
                                       float* dR, double* hist_slot, bool rt_current) {
  FusedPartials fp;
  KT_TRY(fused_launch(ctx, xv, N, L, R, hist_slot, rt_current, &fp));
  k_fused_finish<<<kFsD, 128, 0, ctx->stream>>>(fp, R, dR, &ctx->d_blk->sc);
  KT_LAUNCH_CHECK();
  if (hist_slot != nullptr) KT_TRY(reduce_shards(ctx, hist_slot, 1, KT_F64));
  KT_TRY(reduce_shards(ctx, dR, static_cast<int64_t>(kFsD) * kFsD, KT_F32));
  return KT_OK;
}

// ---------------------------------------------------------- orthogonal step
// E = R^T R - I from the bf16 forms of R^T (rt_hi, rt_lo, which must be current) and, when
// `with_polish`, R <- R - R E / 2 if max|E| > polish_thresh (needs r_hi; refreshes all three forms).
// Every kernel here looks at the device-side gate sc->gate_guard (set by k_step_size or k_force_guard, which also
// clear the running maximum) and does nothing when it is closed.
static kt_status guard(kt_ctx* ctx, const float* R_in, float* R, int d, const WsLayout& L, bool with_polish,
                       float polish_at) {
  Scalars* sc = &ctx->d_blk->sc;
  const int gy = d / 32 < 32 ? d / 32 : 32;
  dim3 lgrid(d / 32, gy), tblock(32, 8);
  k_colnorm_partial<<<lgrid, tblock, 0, ctx->stream>>>(R_in, d, at<float>(ctx, L.colpart), sc);
  KT_LAUNCH_CHECK();
  k_colnorm_final<<<(d + 7) / 8, 256, 0, ctx->stream>>>(at<float>(ctx, L.colpart), d / 32, d, at<float>(ctx, L.diag),
                                                        sc);
  KT_LAUNCH_CHECK();
  const uint64_t ld = static_cast<uint64_t>(d);
  __nv_bfloat16* rt_hi = at<__nv_bfloat16>(ctx, L.rt_hi);
  __nv_bfloat16* rt_lo = at<__nv_bfloat16>(ctx, L.rt_lo);
  __nv_bfloat16* r_hi = at<__nv_bfloat16>(ctx, L.r_hi);
  float* fbuf = at<float>(ctx, L.fbuf);
  {
    GemmParams p = blank_params();
    p.out = fbuf;
    p.ldo = d;
    p.upper_only = 1;  // R^T R is symmetric: tiles below the diagonal are mirrored by k_guard
    p.gate = &sc->gate_guard;
    p.gate_min = 1;
    // (H + L)^T (H + L) without L^T L: that term only matters on the diagonal, which k_guard takes from `diag`
    Operand A[3] = {{rt_hi, ld}, {rt_hi, ld}, {rt_lo, ld}};
    Operand B[3] = {{rt_hi, ld}, {rt_lo, ld}, {rt_hi, ld}};
    KT_TRY(run_gemm<kStoreF32>(ctx, d, d, d, 3, A, B, p, kCatSquare));
  }
  __nv_bfloat16* e_hi = at<__nv_bfloat16>(ctx, L.z_hi);
  k_guard<<<lgrid, tblock, 0, ctx->stream>>>(fbuf, d, (d % 256 == 0) ? 256 : 128, at<float>(ctx, L.diag),
                                             with_polish ? e_hi : nullptr, sc);
  KT_LAUNCH_CHECK();
  if (!with_polish) return KT_OK;
  k_guard_decide<<<1, 1, 0, ctx->stream>>>(sc, polish_at);
  KT_LAUNCH_CHECK();
  {
    GemmParams p = blank_params();
    p.out = fbuf;
    p.ldo = d;
    p.gate = &sc->gate;
    p.gate_min = 1;
    Operand A{r_hi, ld}, B{e_hi, ld};  // (R E)[i][j] = sum_k R[i][k] E[j][k], E symmetric
    KT_TRY(run_gemm<kStoreF32>(ctx, d, d, d, 1, &A, &B, p, kCatSquare));
  }
  k_polish_apply<<<dim3(d / 32, d / 32 < 16 ? d / 32 : 16), tblock, 0, ctx->stream>>>(
      R, fbuf, sc, d, r_hi, rt_hi, rt_lo, L.f16 ? at<__half>(ctx, L.rt16) : nullptr);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

// d <= 512: the whole step and its guard in one cooperative launch (float32 on the CUDA cores).
static bool use_small_orth(const kt_ctx* ctx, int d) { return d <= 512 && ctx->cfg.small_d_orth != 0; }

// run_guard: 1 = measure R^T R - I in this step, 0 = do not, 2 = when the device's drift bound asks for it (and
// then polish already at a quarter of the threshold, as the general path does inside kt_fit).
// parts != null (d == 128): dR is summed inside the launch from the single-pass kernel's partials.
static kt_status small_orth_step_async(kt_ctx* ctx, float* R, const float* dR, int d, float lr, const WsLayout& L,
                                       int run_guard, bool adaptive, const FusedPartials* parts = nullptr,
                                       float* adam_m = nullptr) {
  const kt_config& c = ctx->cfg;
  SmallOrthParams p;
  memset(&p, 0, sizeof(p));
  const size_t dd = static_cast<size_t>(d) * d;
  float* sm = at<float>(ctx, L.small);
  p.R = R;
  p.dR = dR;
  p.d = d;
  p.iters = c.cayley_iters < 0 ? 0 : c.cayley_iters;
  p.gate_terms = c.retract_terms <= 0 ? 1 : 0;
  p.run_guard = run_guard;
  p.lr = lr;
  p.q = c.q;
  p.eps = c.eps;
  p.thresh = c.polish_thresh;
  p.polish_at = (adaptive && c.polish_thresh > 0.f) ? 0.25f * c.polish_thresh : c.polish_thresh;
  if (parts != nullptr) {
    p.use_parts = 1;
    p.fp = *parts;
  }
  p.Rt = sm;
  p.A = sm + dd;
  p.W = sm + 2 * dd;
  p.P0 = sm + 3 * dd;
  p.P1 = sm + 4 * dd;
  p.Rs = sm + 5 * dd;
  p.norm_part = reinterpret_cast<double*>(sm + 6 * dd);
  p.g2_part = p.norm_part + kSoGrid;
  p.max_part = reinterpret_cast<float*>(p.g2_part + kSoGrid);
  p.adam_m = adam_m;
  p.beta1 = c.beta1;
  p.beta2 = c.beta2;
  p.adam_eps = c.adam_eps;
  p.sc = &ctx->d_blk->sc;
  p.r_hi = at<__nv_bfloat16>(ctx, L.r_hi);
  p.rt_hi = at<__nv_bfloat16>(ctx, L.rt_hi);
  p.rt_lo = at<__nv_bfloat16>(ctx, L.rt_lo);
  void* args[] = {&p};
  const void* fn = nullptr;
  switch (d / 128) {
    case 1: fn = reinterpret_cast<const void*>(small_orth_kernel<1>); break;
    case 2: fn = reinterpret_cast<const void*>(small_orth_kernel<2>); break;
    case 3: fn = reinterpret_cast<const void*>(small_orth_kernel<3>); break;
    default: fn = reinterpret_cast<const void*>(small_orth_kernel<4>); break;
  }
  // d == 128: the products stage their second operand (d x d float32) in dynamic shared memory
  const size_t stage_bytes = d == 128 ? dd * sizeof(float) : 0;
  if (stage_bytes > 0) {
    static bool attr_done[kMaxDevices] = {false};
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    const bool cached = ctx->device >= 0 && ctx->device < kMaxDevices;
    if (!cached || !attr_done[ctx->device]) {
      KT_CUDA(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(stage_bytes)));
      if (cached) attr_done[ctx->device] = true;
    }
  }
  // the grid-wide barriers need all kSoGrid CTAs resident at once
  int per_sm = 0;
  KT_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, d, stage_bytes));
  if (per_sm * ctx->sm_count < kSoGrid) return KT_ERR_COOPERATIVE;
  const cudaError_t le = cudaLaunchCooperativeKernel(fn, dim3(kSoGrid), dim3(d), args, stage_bytes, ctx->stream);
  if (le == cudaErrorCooperativeLaunchTooLarge) {
    (void)cudaGetLastError();
    return KT_ERR_COOPERATIVE;
  }
  KT_CUDA(le);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

// One Cayley-SGD step.  `forms_current`: r_hi / rt_hi / rt_lo already hold the bf16 forms of R (true from the
// second step of kt_fit on: the previous step left them).  On return they hold the forms of the new R.
// guard_mode: 1 = measure R^T R - I (and polish if needed) in this step, 2 = do not, 0 = let the device decide from
// its drift bound (see k_step_size).
// adam_m != null: Cayley Adam (momentum buffer; v and the step count live in the device scalar block).
static kt_status orth_step_async(kt_ctx* ctx, float* R, const float* dR, int d, float lr, const WsLayout& L,
                                 int guard_mode, bool forms_current, bool adaptive = false, float* adam_m = nullptr,
                                 bool dr_hi_ready = false) {
  if (use_small_orth(ctx, d))
    return small_orth_step_async(ctx, R, dR, d, lr, L, guard_mode == 1 ? 1 : (guard_mode == 2 ? 0 : 2), adaptive,
                                 nullptr, adam_m);
  const kt_config& c = ctx->cfg;
  Scalars* sc = &ctx->d_blk->sc;
  const uint64_t ld = static_cast<uint64_t>(d);
  const int gy = d / 32 < 32 ? d / 32 : 32;
  dim3 tgrid(d / 32, d / 32), lgrid(d / 32, gy), tblock(32, 8);
  __nv_bfloat16* rt_hi = at<__nv_bfloat16>(ctx, L.rt_hi);
  __nv_bfloat16* rt_lo = at<__nv_bfloat16>(ctx, L.rt_lo);
  __nv_bfloat16* r_hi = at<__nv_bfloat16>(ctx, L.r_hi);
  __nv_bfloat16* z_hi = at<__nv_bfloat16>(ctx, L.z_hi);
  __nv_bfloat16* w_hi = at<__nv_bfloat16>(ctx, L.w_hi);
  __nv_bfloat16* w_lo = at<__nv_bfloat16>(ctx, L.w_lo);
  float* fbuf = at<float>(ctx, L.fbuf);
  const int cfg_terms = c.retract_terms < 0 ? 0 : (c.retract_terms > 3 ? 3 : c.retract_terms);  // 0 = automatic
  const int max_terms = cfg_terms > 0 ? cfg_terms : 2;
  const int s = c.cayley_iters < 0 ? 0 : c.cayley_iters;

  // A = dR R^T (the gradient needs no more than bf16), W = (A - A^T)/2, alpha and the step's gates
  if (adam_m) {
    // Cayley Adam: the direction comes from the momentum M <- beta1 M + (1 - beta1) dR, scaled by 1/r
    k_adam_moment<<<tgrid, tblock, 0, ctx->stream>>>(adam_m, dR, c.beta1, d, z_hi, at<double>(ctx, L.norm_blocks));
    KT_LAUNCH_CHECK();
    k_adam_scalars<<<1, 1024, 0, ctx->stream>>>(at<double>(ctx, L.norm_blocks), L.norm_n, c.beta1, c.beta2, c.adam_eps,
                                                sc);
    KT_LAUNCH_CHECK();
  } else if (!dr_hi_ready) {  // (inside kt_fit the split-K sum of the gradient has already left bf16(dR) in z_hi)
    k_split_bf16<false><<<tgrid, tblock, 0, ctx->stream>>>(dR, d, z_hi /* dR hi: free until P^T is written */,
                                                           nullptr, d);
    KT_LAUNCH_CHECK();
  }
  if (!forms_current) {
    k_split_r<<<tgrid, tblock, 0, ctx->stream>>>(R, d, r_hi, rt_hi, rt_lo);
    KT_LAUNCH_CHECK();
  }
  {
    GemmParams p = blank_params();
    p.out = fbuf;
    p.ldo = d;
    Operand A{z_hi, ld}, B{r_hi, ld};
    KT_TRY(run_gemm<kStoreF32>(ctx, d, d, d, 1, &A, &B, p, kCatSquare));
  }
  k_skew<<<tgrid, tblock, 0, ctx->stream>>>(fbuf, d, w_hi, max_terms == 3 ? w_lo : nullptr,
                                            at<double>(ctx, L.norm_blocks), adam_m ? sc : nullptr);
  KT_LAUNCH_CHECK();
  // a short power iteration on W^T W = -W^2 (W is skew): v <- W v, 2 * norm_iters times from a fixed +-1 vector;
  // the growth of the last application estimates ||W||_2 for the step's decisions (not for alpha)
  const float* pv_prev = nullptr;
  const float* pv_last = nullptr;
  const int n_mv = c.norm_iters > 0 ? 2 * (c.norm_iters > 16 ? 16 : c.norm_iters) : 0;
  if (n_mv > 0) {
    // (the products return at once when ||W||_F alone already gives the cheapest step: see k_w_norm)
    k_w_norm<<<1, 1024, 0, ctx->stream>>>(at<double>(ctx, L.norm_blocks), L.norm_n, lr, c.q, c.eps, s, sc);
    KT_LAUNCH_CHECK();
    float* pv[2] = {at<float>(ctx, L.pvec), at<float>(ctx, L.pvec) + d};
    for (int i = 0; i < n_mv; ++i) {
      k_skew_matvec<<<d / 8, 256, 0, ctx->stream>>>(w_hi, d, i == 0 ? nullptr : pv[(i + 1) & 1], pv[i & 1], sc);
      KT_LAUNCH_CHECK();
    }
    pv_prev = pv[n_mv & 1];        // written by application n_mv - 2
    pv_last = pv[(n_mv + 1) & 1];  // written by application n_mv - 1
  }
  k_step_size<<<1, 1024, 0, ctx->stream>>>(at<double>(ctx, L.norm_blocks), n_mv > 0 ? 0 : L.norm_n, lr, c.q, c.eps, sc,
                                          d, s, cfg_terms, cfg_terms == 0 ? 1 : 0, guard_mode, c.polish_thresh,
                                          pv_prev, pv_last);
  KT_LAUNCH_CHECK();

  // P_0 = W R with R^T as a bf16 split (it multiplies alpha directly; the device picks one or two terms);
  // P_{k+1} = W P_k with P_k^T in plain bf16 (these terms carry alpha^2 and higher), skipped on the device once
  // they are below float32 resolution.  (W Z)[i][j] = sum_k W[i][k] Zt[j][k].
  for (int k = 0; k <= s; ++k) {
    GemmParams p = blank_params();
    p.out = fbuf;
    p.ldo = d;
    if (k == 0) {
      p.terms_dev = &sc->p0_terms;
      Operand A[3] = {{w_hi, ld}, {w_hi, ld}, {w_lo, ld}};
      Operand B[3] = {{rt_hi, ld}, {rt_lo, ld}, {rt_hi, ld}};
      KT_TRY(run_gemm<kStoreF32>(ctx, d, d, d, max_terms, A, B, p, kCatSquare));
    } else {
      p.gate = &sc->n_terms;
      p.gate_min = static_cast<unsigned int>(k + 1);
      Operand A{w_hi, ld}, B{z_hi, ld};
      KT_TRY(run_gemm<kStoreF32>(ctx, d, d, d, 1, &A, &B, p, kCatSquare));
    }
    k_series_term<<<lgrid, tblock, 0, ctx->stream>>>(R, fbuf, sc, k, d, z_hi, r_hi, rt_hi, rt_lo,
                                                     k == 0 ? adam_m : nullptr,
                                                     L.f16 ? at<__half>(ctx, L.rt16) : nullptr);
    KT_LAUNCH_CHECK();
  }
  if (guard_mode != 2) {
    const float th = ctx->cfg.polish_thresh;
    KT_TRY(guard(ctx, R, R, d, L, true, (adaptive && th > 0.f) ? 0.25f * th : th));
  }
  return KT_OK;
}

// Copies the scalar block back and synchronises; maps a recorded wait time-out.
static kt_status sync_scalars(kt_ctx* ctx) {
  KT_CUDA(cudaMemcpyAsync(&ctx->h_blk->sc, &ctx->d_blk->sc, sizeof(Scalars), cudaMemcpyDeviceToHost, ctx->stream));
  KT_CUDA(cudaStreamSynchronize(ctx->stream));
  if (ctx->h_blk->sc.err_word != 0) {
    (void)cudaMemsetAsync(&ctx->d_blk->sc.err_word, 0, sizeof(unsigned int), ctx->stream);
    return KT_ERR_TIMEOUT;
  }
  return KT_OK;
}

static kt_status check_d(int64_t d) {
  if (d < 128 || d % 128 != 0 || d > 65536) return KT_ERR_SHAPE;
  return KT_OK;
}

// A rotation shared by several equally shaped activation buffers: every step works on a minibatch of `batch`
// samples (runs of `rps` consecutive rows) named by `order` (host; steps * batch ids, id = buffer * samples per
// buffer + sample within the buffer).
struct SharedSrc {
  const kt_mat* bufs;
  int n_bufs;
  int64_t rps;
  const int32_t* order;
  int batch;
};

// X is the calibration matrix, or (sh != null) the first of the shared buffers, which stands for their common shape.
static kt_status fit_impl(kt_ctx* ctx, const kt_mat& X, float* R, int32_t steps, float lr, kt_fit_report* report,
                          const SharedSrc* sh = nullptr) {
  int64_t N64, d64;
  KT_TRY(check_x(X, &N64, &d64));
  if (R == nullptr || steps < 0) return KT_ERR_INVALID_ARG;
  if (!aligned16(R)) return KT_ERR_ALIGN;
  const bool adam = ctx->cfg.optimizer == 1;
  const int spb = sh ? static_cast<int>(N64 / sh->rps) : 0;  // samples per buffer
  if (sh) N64 = static_cast<int64_t>(sh->batch) * sh->rps;
  const WsLayout L = make_layout(N64, d64, X.dtype, &ctx->cfg, sh ? sh->batch : 0);
  KT_TRY(check_ws(ctx, L));
  const int N = static_cast<int>(N64), d = static_cast<int>(d64);
  if (sh) {
    const void* bases[kMaxSharedBufs];
    for (int b = 0; b < sh->n_bufs; ++b) bases[b] = sh->bufs[b].data;
    KT_CUDA(cudaMemcpyAsync(ctx->ws + L.gather_bases, bases, sizeof(void*) * sh->n_bufs, cudaMemcpyHostToDevice,
                            ctx->stream));
    KT_CUDA(cudaStreamSynchronize(ctx->stream));  // `bases` is a stack array
  }
  float* adam_m = nullptr;
  if (adam) {  // every fit starts Cayley Adam from a zero state
    adam_m = at<float>(ctx, L.adam_m);
    KT_CUDA(cudaMemsetAsync(adam_m, 0, static_cast<size_t>(d) * d * 4, ctx->stream));
    k_adam_set<<<1, 1, 0, ctx->stream>>>(&ctx->d_blk->sc, 0.0, 0u);
    KT_LAUNCH_CHECK();
  }
  k_fit_begin<<<1, 1, 0, ctx->stream>>>(&ctx->d_blk->sc);
  KT_LAUNCH_CHECK();
  XView xv;
  memset(&xv, 0, sizeof(xv));
  const bool fused = use_fused(ctx, d);
  if (!sh) {
    if (fused) {
      KT_TRY(fused_encode(ctx, X, L, &xv));
    } else {
      KT_TRY(ingest_x_full(ctx, X, L, &xv));
    }
  }
  float* dR = at<float>(ctx, L.dr);
  // the Cayley step's first product reads bf16(dR): when the gradient ends in a split-K sum, that sum writes it too
  // (not in a sharded fit: there the sum over shards changes dR after the split-K sum)
  __nv_bfloat16* dr_hi = (!fused && !adam && !use_small_orth(ctx, d) && plan_split_k(d, N).splits > 1 &&
                          ctx->reduce_fn == nullptr)
                             ? at<__nv_bfloat16>(ctx, L.z_hi)
                             : nullptr;
  const int ge = ctx->cfg.guard_every < 1 ? 1 : ctx->cfg.guard_every;
  double first = 0.0, last = 0.0;
  int done = 0;
  for (int k = 0; k < steps; ++k) {
    const int slot = k % kHistMax;
    if (k > 0 && slot == 0) {
      // history block full: bring it to the host before it is overwritten
      KT_CUDA(cudaMemcpyAsync(ctx->h_blk->hist, ctx->d_blk->hist, sizeof(double) * kHistMax, cudaMemcpyDeviceToHost,
                              ctx->stream));
      KT_CUDA(cudaStreamSynchronize(ctx->stream));
      if (k == kHistMax) first = ctx->h_blk->hist[0];
      if (report && report->loss_history)
        memcpy(report->loss_history + (k - kHistMax), ctx->h_blk->hist, sizeof(double) * kHistMax);
    }
    if (sh) {
      // this step's minibatch: gather its samples into the dense bf16 matrix, normalise, transpose
      const int cslot = k % kIdsChunk;
      if (cslot == 0) {
        const int n_steps = (steps - k < kIdsChunk) ? steps - k : kIdsChunk;
        if (k > 0) KT_CUDA(cudaStreamSynchronize(ctx->stream));  // the previous chunk's ids are still being read
        KT_CUDA(cudaMemcpyAsync(ctx->ws + L.gather_ids, sh->order + static_cast<size_t>(k) * sh->batch,
                                sizeof(int32_t) * n_steps * sh->batch, cudaMemcpyHostToDevice, ctx->stream));
      }
      __nv_bfloat16* xb = at<__nv_bfloat16>(ctx, L.xb);
      const void* const* bases = at<const void*>(ctx, L.gather_bases);
      const int* ids = at<int>(ctx, L.gather_ids) + static_cast<size_t>(cslot) * sh->batch;
      const int rps = static_cast<int>(sh->rps);
      const bool norm = ctx->cfg.rmsnorm != 0 && !fused;
      xv.row_scale = nullptr;
      if (fused) {
        // gather straight into the single-pass kernel's encoding (row-normalised float16 and the rows' mean squares)
        float* ms = at<float>(ctx, L.rowscale);
        __half* x16 = reinterpret_cast<__half*>(xb);
        const unsigned eg = static_cast<unsigned>((N + 15) / 16);
        if (X.dtype == KT_BF16)
          k_encode_rows_128<__nv_bfloat16><<<eg, 256, 0, ctx->stream>>>(nullptr, X.ld, N, x16, ms, bases, spb, rps, ids);
        else
          k_encode_rows_128<float><<<eg, 256, 0, ctx->stream>>>(nullptr, X.ld, N, x16, ms, bases, spb, rps, ids);
        xv.row_ms = ms;
      } else if (L.f16 && X.dtype == KT_BF16) {
        // float16 forward operands: the samples' rows go straight into that encoding (with the RMSNorm factors when
        // asked for) and, below, into the transpose; no dense bf16 copy of the minibatch is made
        float* rsc = norm ? at<float>(ctx, L.rowscale) : nullptr;
        k_gather_encode_rows_f16<<<N, 256, 0, ctx->stream>>>(bases, X.ld, spb, rps, ids, d, ctx->cfg.rms_eps, rsc,
                                                             at<__half>(ctx, L.x16), at<float>(ctx, L.rowacc));
        xv.row_scale = rsc;
      } else if (norm) {
        // gather and RMSNorm factors in one pass over the samples' rows
        float* rsc = at<float>(ctx, L.rowscale);
        if (X.dtype == KT_BF16)
          k_row_scale<__nv_bfloat16><<<N, 256, 0, ctx->stream>>>(nullptr, X.ld, d, ctx->cfg.rms_eps, rsc, xb, bases,
                                                                 spb, rps, ids);
        else
          k_row_scale<float><<<N, 256, 0, ctx->stream>>>(nullptr, X.ld, d, ctx->cfg.rms_eps, rsc, xb, bases, spb, rps,
                                                         ids);
        xv.row_scale = rsc;
      } else if (X.dtype == KT_BF16) {
        k_gather_samples<__nv_bfloat16><<<N, 256, 0, ctx->stream>>>(bases, X.ld, spb, rps, ids, d, xb);
      } else {
        k_gather_samples<float><<<N, 256, 0, ctx->stream>>>(bases, X.ld, spb, rps, ids, d, xb);
      }
      KT_LAUNCH_CHECK();
      xv.xb = xb;
      xv.ldx = d;
      if (!fused && L.f16 && X.dtype == KT_BF16) {
        dim3 tg(d / 128, (N + 63) / 64);
        k_transpose_x_bf16<<<tg, 256, 0, ctx->stream>>>(nullptr, X.ld, N, d, at<__nv_bfloat16>(ctx, L.xt), L.ldt,
                                                        bases, spb, rps, ids);
        KT_LAUNCH_CHECK();
        xv.xb = nullptr;   // (not made; the forward pass reads the encoding)
        xv.x16 = at<__half>(ctx, L.x16);
        xv.acc_scale = at<float>(ctx, L.rowacc);
      } else if (!fused) {  // the token GEMM of the backward pass reads the transpose
        KT_TRY(transpose_x_bf16(ctx, xb, d, N, d, L));
        KT_TRY(finish_view(ctx, N, d, L, &xv));   // (and the forward pass, maybe, the float16 encoding)
      }
    }
    // from the second step on, the previous step left the bf16 forms of R in the workspace
    // d = 128 with the one-launch orthogonal step: that launch also sums the single-pass kernel's partials
    const bool fold = fused && use_small_orth(ctx, d) && ctx->reduce_fn == nullptr;
    FusedPartials parts;
    // (that launch also leaves the bf16 forms of the new Rc^T; any other step leaves those of R^T, so the
    // single-pass kernel's operand is then made afresh)
    if (fold)
      KT_TRY(fused_launch(ctx, xv, N, L, R, &ctx->d_blk->hist[slot], k > 0, &parts));
    else if (fused)
      KT_TRY(fused_loss_grad_async(ctx, xv, N, L, R, dR, &ctx->d_blk->hist[slot], false));
    else
      KT_TRY(loss_grad_async(ctx, xv, N, d, L, R, dR, &ctx->d_blk->hist[slot], k > 0, dr_hi));
    // guard: a fixed cadence when guard_every >= 1; otherwise measured on the first and the last step and in between
    // whenever the device's drift bound asks for it
    int guard_mode;
    if (ctx->cfg.guard_every >= 1)
      guard_mode = (((k + 1) % ge == 0) || (k + 1 == steps)) ? 1 : 2;
    else
      guard_mode = (k == 0 || k + 1 == steps) ? 1 : 0;
    if (fold)
      KT_TRY(small_orth_step_async(ctx, R, dR, d, lr, L, guard_mode == 1 ? 1 : (guard_mode == 2 ? 0 : 2),
                                   ctx->cfg.guard_every < 1, &parts, adam_m));
    else
      // (the single-pass kernel has put the forms of Rc^T where the step expects those of R^T: not current then)
      KT_TRY(orth_step_async(ctx, R, dR, d, lr, L, guard_mode, k > 0 && !fused, ctx->cfg.guard_every < 1, adam_m,
                             dr_hi != nullptr));
    done = k + 1;
  }
  if (steps > 0) {
    const int tail = (steps - 1) % kHistMax + 1;  // entries of the last history block
    KT_CUDA(cudaMemcpyAsync(ctx->h_blk->hist, ctx->d_blk->hist, sizeof(double) * tail, cudaMemcpyDeviceToHost,
                            ctx->stream));
  }
  kt_status st = sync_scalars(ctx);
  if (steps > 0) {
    const int tail = (steps - 1) % kHistMax + 1;
    if (steps <= kHistMax) first = ctx->h_blk->hist[0];
    last = ctx->h_blk->hist[tail - 1];
    if (report && report->loss_history)
      memcpy(report->loss_history + (steps - tail), ctx->h_blk->hist, sizeof(double) * tail);
  }
  if (report) {
    report->steps_done = done;
    report->degenerate_rows = static_cast<int32_t>(ctx->h_blk->sc.deg_rows);
    report->loss_first = first;
    report->loss_last = last;
    report->orth_err = static_cast<double>(__builtin_bit_cast(float, ctx->h_blk->sc.max_e_bits));
    report->alpha_last = ctx->h_blk->sc.alpha;
    report->w_norm_last = ctx->h_blk->sc.wnorm;
    report->w_op_last = ctx->h_blk->sc.wop;
    report->series_terms_last = static_cast<int32_t>(ctx->h_blk->sc.n_terms);
    report->p0_terms_last = static_cast<int32_t>(ctx->h_blk->sc.p0_terms);
    report->guards_run = static_cast<int32_t>(ctx->h_blk->sc.guards);
  }
  if (st != KT_OK) return st;
  if (steps > 0 && !isfinite(last)) return KT_ERR_NONFINITE;
  return KT_OK;
}

}  // namespace kt

using namespace kt;

// ============================================================== C ABI
extern "C" {

void kt_default_config(kt_config* cfg) {
  if (!cfg) return;
  memset(cfg, 0, sizeof(*cfg));
  cfg->kappa_target = 1.8f;
  cfg->cayley_iters = 2;
  cfg->q = 0.5f;
  cfg->eps = 1e-8f;
  cfg->polish_thresh = 1e-5f;
  cfg->retract_terms = 0;
  cfg->guard_every = 0;
  cfg->forward_terms = 0;
  cfg->small_d_fused = 1;
  cfg->small_d_orth = 1;
  cfg->optimizer = 0;
  cfg->beta1 = 0.9f;
  cfg->beta2 = 0.99f;
  cfg->adam_eps = 1e-8f;
  cfg->norm_iters = 2;
  cfg->backward_mode = 0;
  cfg->forward_bf16 = 0;
  cfg->cta_pairs = 1;
  cfg->loss_mode = 0;
  cfg->rmsnorm = 0;
  cfg->rms_eps = 1e-6f;
  cfg->wait_limit_ms = 4000;
}

const char* kt_status_string(kt_status s) {
  switch (s) {
    case KT_OK: return "ok";
    case KT_ERR_INVALID_ARG: return "invalid argument";
    case KT_ERR_SHAPE: return "unsupported shape";
    case KT_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
    case KT_ERR_WORKSPACE: return "workspace missing or too small";
    case KT_ERR_ARCH: return "device is not sm_100";
    case KT_ERR_CUDA: return "CUDA call failed";
    case KT_ERR_NONFINITE: return "non-finite loss";
    case KT_ERR_TIMEOUT: return "device-side wait timed out";
    case KT_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
    case KT_ERR_COOPERATIVE: return "the one-launch step for d <= 512 needs 128 co-resident CTAs (set small_d_orth = 0)";
    case KT_ERR_REDUCE: return "the caller's reduce hook reported a failure";
  }
  return "unknown status";
}

kt_status kt_create(kt_ctx** out, const kt_config* cfg, void* cuda_stream) {
  if (!out) return KT_ERR_INVALID_ARG;
  *out = nullptr;
  int dev = 0;
  KT_CUDA(cudaGetDevice(&dev));
  int major = 0, sms = 0;
  KT_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  KT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (major != 10) return KT_ERR_ARCH;
  kt_ctx* c = new (std::nothrow) kt_ctx;
  if (!c) return KT_ERR_CUDA;
  memset(c, 0, sizeof(*c));
  if (cfg) c->cfg = *cfg; else kt_default_config(&c->cfg);
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->device = dev;
  c->sm_count = sms;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete c;
    return KT_ERR_CUDA;
  }
  c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&c->d_blk, sizeof(DeviceBlock)) != cudaSuccess) {
    delete c;
    return KT_ERR_CUDA;
  }
  if (cudaMallocHost(&c->h_blk, sizeof(DeviceBlock)) != cudaSuccess) {
    cudaFree(c->d_blk);
    delete c;
    return KT_ERR_CUDA;
  }
  if (cudaMemset(c->d_blk, 0, sizeof(DeviceBlock)) != cudaSuccess) {
    cudaFreeHost(c->h_blk);
    cudaFree(c->d_blk);
    delete c;
    return KT_ERR_CUDA;
  }
  memset(c->h_blk, 0, sizeof(DeviceBlock));
  *out = c;
  return KT_OK;
}

void kt_destroy(kt_ctx* ctx) {
  if (!ctx) return;
  cudaStreamSynchronize(ctx->stream);
  if (ctx->prof_ev) {
    for (int i = 0; i < 2 * kProfPairs; ++i) cudaEventDestroy(ctx->prof_ev[i]);
    delete[] ctx->prof_ev;
    delete[] ctx->prof_cat;
  }
  cudaFreeHost(ctx->h_blk);
  cudaFree(ctx->d_blk);
  delete ctx;
}

kt_status kt_workspace_bytes(const kt_ctx* ctx, int64_t N, int64_t d, int32_t x_dtype, size_t* bytes) {
  if (!bytes) return KT_ERR_INVALID_ARG;
  if (x_dtype != KT_BF16 && x_dtype != KT_F32) return KT_ERR_INVALID_ARG;
  if (N < 1 || N > 0x7fffff00ll) return KT_ERR_SHAPE;
  KT_TRY(check_d(d));
  *bytes = make_layout(N, d, x_dtype, ctx ? &ctx->cfg : nullptr).total;
  return KT_OK;
}

kt_status kt_set_workspace(kt_ctx* ctx, void* dev_ptr, size_t bytes) {
  if (!ctx) return KT_ERR_INVALID_ARG;
  if (dev_ptr != nullptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255u) != 0) return KT_ERR_ALIGN;
  ctx->ws = static_cast<uint8_t*>(dev_ptr);
  ctx->ws_bytes = dev_ptr ? bytes : 0;
  return KT_OK;
}

kt_status kt_init_rotation(kt_ctx* ctx, float* R, int64_t d, int32_t kind) {
  if (!ctx || !R || (kind != 0 && kind != 1)) return KT_ERR_INVALID_ARG;
  if (d < 1 || d > 65536) return KT_ERR_SHAPE;
  if (kind == 1 && (d & (d - 1)) != 0) return KT_ERR_SHAPE;
  const float scale = static_cast<float>(1.0 / sqrt(static_cast<double>(d)));
  const long long n = d * d;
  k_init_rotation<<<static_cast<unsigned>((n + 255) / 256), 256, 0, ctx->stream>>>(R, static_cast<int>(d), kind, scale);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

kt_status kt_kurtosis_loss(kt_ctx* ctx, kt_mat X, const float* R, double* loss) {
  if (!ctx || !R || !loss) return KT_ERR_INVALID_ARG;
  int64_t N, d;
  KT_TRY(check_x(X, &N, &d));
  if (!aligned16(R)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N, d, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  XView xv;
  KT_TRY(ingest_x_forward(ctx, X, L, &xv));
  KT_TRY(cast_rt(ctx, R, static_cast<int>(d), N, L));
  KT_TRY(forward_loss(ctx, xv, static_cast<int>(N), static_cast<int>(d), L, nullptr));
  KT_TRY(sync_scalars(ctx));
  *loss = ctx->h_blk->sc.loss;
  return isfinite(*loss) ? KT_OK : KT_ERR_NONFINITE;
}

kt_status kt_row_moments(kt_ctx* ctx, kt_mat X, const float* R, float* moments) {
  if (!ctx || !R || !moments) return KT_ERR_INVALID_ARG;
  int64_t N, d;
  KT_TRY(check_x(X, &N, &d));
  if (!aligned16(R) || !aligned16(moments)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N, d, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  XView xv;
  KT_TRY(ingest_x_forward(ctx, X, L, &xv));
  KT_TRY(cast_rt(ctx, R, static_cast<int>(d), N, L));
  KT_TRY(forward_loss(ctx, xv, static_cast<int>(N), static_cast<int>(d), L, nullptr));
  KT_CUDA(cudaMemcpyAsync(moments, at<float4>(ctx, L.moments), static_cast<size_t>(N) * 16, cudaMemcpyDeviceToDevice,
                          ctx->stream));
  return KT_OK;
}

kt_status kt_rotate(kt_ctx* ctx, kt_mat X, const float* R, float* Y) {
  if (!ctx || !R || !Y) return KT_ERR_INVALID_ARG;
  int64_t N, d;
  KT_TRY(check_x(X, &N, &d));
  if (!aligned16(R) || !aligned16(Y)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N, d, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  XView xv;
  KT_TRY(ingest_x_forward(ctx, X, L, &xv));
  KT_TRY(cast_rt(ctx, R, static_cast<int>(d), N, L));
  GemmParams p = blank_params();
  p.out = Y;
  p.ldo = d;
  const FwdOperands f = fwd_operands(ctx, xv, static_cast<int>(d), N, L, &p);
  return run_gemm<kStoreF32>(ctx, static_cast<int>(N), static_cast<int>(d), static_cast<int>(d), f.terms, f.A, f.B, p,
                             kCatForward);
}

kt_status kt_loss_grad(kt_ctx* ctx, kt_mat X, const float* R, float* dR, double* loss) {
  if (!ctx || !R || !dR) return KT_ERR_INVALID_ARG;
  int64_t N, d;
  KT_TRY(check_x(X, &N, &d));
  if (!aligned16(R) || !aligned16(dR)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N, d, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  XView xv;
  if (use_fused(ctx, static_cast<int>(d))) {
    KT_TRY(fused_encode(ctx, X, L, &xv));
    KT_TRY(fused_loss_grad_async(ctx, xv, static_cast<int>(N), L, R, dR, nullptr, false));
  } else {
    KT_TRY(ingest_x_full(ctx, X, L, &xv));
    KT_TRY(loss_grad_async(ctx, xv, static_cast<int>(N), static_cast<int>(d), L, R, dR, nullptr, false));
  }
  if (!loss) return KT_OK;
  KT_TRY(sync_scalars(ctx));
  *loss = ctx->h_blk->sc.loss;
  return isfinite(*loss) ? KT_OK : KT_ERR_NONFINITE;
}

kt_status kt_orth_step(kt_ctx* ctx, float* R, const float* dR, int64_t d, float lr) {
  if (!ctx || !R || !dR || !(lr >= 0.f)) return KT_ERR_INVALID_ARG;
  KT_TRY(check_d(d));
  if (!aligned16(R) || !aligned16(dR)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(1, d, KT_BF16, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  return orth_step_async(ctx, R, dR, static_cast<int>(d), lr, L, 1, false);
}

kt_status kt_adam_step(kt_ctx* ctx, float* R, const float* dR, float* M, kt_adam_state* st, int64_t d, float lr) {
  if (!ctx || !R || !dR || !M || !st || !(lr >= 0.f) || st->step < 0 || !(st->v >= 0.0)) return KT_ERR_INVALID_ARG;
  const kt_config& c = ctx->cfg;
  if (!(c.beta1 >= 0.f && c.beta1 < 1.f) || !(c.beta2 >= 0.f && c.beta2 < 1.f) || !(c.adam_eps > 0.f))
    return KT_ERR_INVALID_ARG;
  KT_TRY(check_d(d));
  if (!aligned16(R) || !aligned16(dR) || !aligned16(M)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(1, d, KT_BF16, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  k_adam_set<<<1, 1, 0, ctx->stream>>>(&ctx->d_blk->sc, st->v, static_cast<unsigned int>(st->step));
  KT_LAUNCH_CHECK();
  KT_TRY(orth_step_async(ctx, R, dR, static_cast<int>(d), lr, L, 1, false, false, M));
  KT_TRY(sync_scalars(ctx));
  st->v = ctx->h_blk->sc.adam_v;
  st->step = static_cast<int32_t>(ctx->h_blk->sc.adam_k);
  return KT_OK;
}

kt_status kt_orth_error(kt_ctx* ctx, const float* R, int64_t d, double* err) {
  if (!ctx || !R || !err) return KT_ERR_INVALID_ARG;
  KT_TRY(check_d(d));
  if (!aligned16(R)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(1, d, KT_BF16, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  dim3 tgrid(static_cast<unsigned>(d / 32), static_cast<unsigned>(d / 32)), tblock(32, 8);
  k_split_bf16<true><<<tgrid, tblock, 0, ctx->stream>>>(R, d, at<__nv_bfloat16>(ctx, L.rt_hi),
                                                        at<__nv_bfloat16>(ctx, L.rt_lo), d);
  KT_LAUNCH_CHECK();
  k_force_guard<<<1, 1, 0, ctx->stream>>>(&ctx->d_blk->sc);
  KT_LAUNCH_CHECK();
  KT_TRY(guard(ctx, R, nullptr, static_cast<int>(d), L, false, 0.f));
  KT_TRY(sync_scalars(ctx));
  *err = static_cast<double>(__builtin_bit_cast(float, ctx->h_blk->sc.max_e_bits));
  return KT_OK;
}

kt_status kt_fit(kt_ctx* ctx, kt_mat X, float* R, int32_t steps, float lr, kt_fit_report* report) {
  if (!ctx || !(lr >= 0.f)) return KT_ERR_INVALID_ARG;
  return fit_impl(ctx, X, R, steps, lr, report);
}

// the caller's reduce hook and the batch's row count stay attached to the context for the duration of one fit
struct ShardScope {
  kt_ctx* ctx;
  ShardScope(kt_ctx* c, kt_reduce_fn fn, void* user, int64_t rows_total) : ctx(c) {
    c->reduce_fn = fn;
    c->reduce_user = user;
    c->rows_total = static_cast<double>(rows_total);
  }
  ~ShardScope() {
    ctx->reduce_fn = nullptr;
    ctx->reduce_user = nullptr;
    ctx->rows_total = 0.0;
  }
};

kt_status kt_fit_sharded(kt_ctx* ctx, kt_mat X_local, float* R, int64_t rows_total, kt_reduce_fn reduce, void* user,
                         int32_t steps, float lr, kt_fit_report* report) {
  if (!ctx || !(lr >= 0.f) || rows_total < X_local.rows) return KT_ERR_INVALID_ARG;
  ShardScope scope(ctx, reduce, user, rows_total);
  return fit_impl(ctx, X_local, R, steps, lr, report);
}

kt_status kt_test_wait_timeout(kt_ctx* ctx, int32_t limit_ms) {
  if (!ctx || limit_ms < 1 || limit_ms > 1000) return KT_ERR_INVALID_ARG;
  k_wait_probe<<<1, 32, 0, ctx->stream>>>(static_cast<unsigned long long>(limit_ms) * 1000000ull,
                                          &ctx->d_blk->sc.err_word);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

kt_status kt_fit_layers(kt_ctx* ctx, const kt_mat* X_layers, float* const* R_layers, int32_t L, int32_t first_layer,
                        int32_t steps, float lr, kt_fit_report* per_layer) {
  if (!ctx || !X_layers || !R_layers || L < 0 || first_layer < 0 || first_layer > L || !(lr >= 0.f))
    return KT_ERR_INVALID_ARG;
  // validate every layer before touching any
  for (int l = first_layer; l < L; ++l) {
    int64_t N, d;
    KT_TRY(check_x(X_layers[l], &N, &d));
    if (R_layers[l] == nullptr) return KT_ERR_INVALID_ARG;
    if (!aligned16(R_layers[l])) return KT_ERR_ALIGN;
    if (X_layers[l].rows != X_layers[first_layer].rows || X_layers[l].cols != X_layers[first_layer].cols ||
        X_layers[l].dtype != X_layers[first_layer].dtype)
      return KT_ERR_SHAPE;
  }
  for (int l = first_layer; l < L; ++l) {
    KT_TRY(fit_impl(ctx, X_layers[l], R_layers[l], steps, lr, per_layer ? &per_layer[l] : nullptr));
  }
  return KT_OK;
}

kt_status kt_fit_shared_workspace_bytes(const kt_ctx* ctx, int64_t rows_per_sample, int32_t batch, int64_t d,
                                        size_t* bytes) {
  if (!ctx || !bytes) return KT_ERR_INVALID_ARG;
  if (rows_per_sample < 1 || batch < 1 || batch > 65536 || rows_per_sample * batch > 0x7fffff00ll) return KT_ERR_SHAPE;
  KT_TRY(check_d(d));
  *bytes = make_layout(rows_per_sample * batch, d, KT_BF16, &ctx->cfg, batch).total;
  return KT_OK;
}

kt_status kt_fit_shared(kt_ctx* ctx, const kt_mat* X_bufs, int32_t n_bufs, int64_t rows_per_sample,
                        const int32_t* order, int32_t batch, float* R, int32_t steps, float lr,
                        kt_fit_report* report) {
  if (!ctx || !X_bufs || !order || !R || n_bufs < 1 || n_bufs > kMaxSharedBufs || steps < 0 || !(lr >= 0.f))
    return KT_ERR_INVALID_ARG;
  if (rows_per_sample < 1 || batch < 1 || batch > 65536 || rows_per_sample * batch > 0x7fffff00ll) return KT_ERR_SHAPE;
  int64_t N0, d0;
  KT_TRY(check_x(X_bufs[0], &N0, &d0));
  if (N0 % rows_per_sample != 0) return KT_ERR_SHAPE;
  for (int b = 1; b < n_bufs; ++b) {
    int64_t N, d;
    KT_TRY(check_x(X_bufs[b], &N, &d));
    if (N != N0 || d != d0 || X_bufs[b].dtype != X_bufs[0].dtype || X_bufs[b].ld != X_bufs[0].ld) return KT_ERR_SHAPE;
  }
  const int64_t n_samples = static_cast<int64_t>(n_bufs) * (N0 / rows_per_sample);
  for (int64_t i = 0; i < static_cast<int64_t>(steps) * batch; ++i)
    if (order[i] < 0 || order[i] >= n_samples) return KT_ERR_INVALID_ARG;
  SharedSrc sh{X_bufs, n_bufs, rows_per_sample, order, batch};
  return fit_impl(ctx, X_bufs[0], R, steps, lr, report, &sh);
}

kt_status kt_fit_shared_sharded(kt_ctx* ctx, const kt_mat* X_bufs, int32_t n_bufs, int64_t rows_per_sample,
                                const int32_t* order, int32_t batch, float* R, int64_t rows_total,
                                kt_reduce_fn reduce, void* user, int32_t steps, float lr, kt_fit_report* report) {
  if (!ctx || rows_total < static_cast<int64_t>(batch) * rows_per_sample) return KT_ERR_INVALID_ARG;
  ShardScope scope(ctx, reduce, user, rows_total);
  return kt_fit_shared(ctx, X_bufs, n_bufs, rows_per_sample, order, batch, R, steps, lr, report);
}

kt_status kt_fit_host(kt_ctx* ctx, kt_mat X_host, void* X_dev_staging, float* R_host, float* R_dev, int32_t steps,
                      float lr, kt_fit_report* report) {
  if (!ctx || !X_dev_staging || !R_host || !R_dev || !(lr >= 0.f) || steps < 0) return KT_ERR_INVALID_ARG;
  kt_mat Xd = X_host;
  Xd.data = X_dev_staging;
  int64_t N, d;
  KT_TRY(check_x(Xd, &N, &d));
  if (X_host.data == nullptr) return KT_ERR_INVALID_ARG;
  if (!aligned16(R_dev)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N, d, Xd.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  const size_t es = (Xd.dtype == KT_BF16) ? 2 : 4;
  KT_CUDA(cudaMemcpyAsync(X_dev_staging, X_host.data, static_cast<size_t>(N) * Xd.ld * es, cudaMemcpyHostToDevice,
                          ctx->stream));
  KT_CUDA(cudaMemcpyAsync(R_dev, R_host, static_cast<size_t>(d) * d * 4, cudaMemcpyHostToDevice, ctx->stream));
  kt_status st = fit_impl(ctx, Xd, R_dev, steps, lr, report);
  KT_CUDA(cudaMemcpyAsync(R_host, R_dev, static_cast<size_t>(d) * d * 4, cudaMemcpyDeviceToHost, ctx->stream));
  KT_CUDA(cudaStreamSynchronize(ctx->stream));
  return st;
}

// levels of a k-bit quantizer: symmetric codes in [-(2^(k-1) - 1), 2^(k-1) - 1], asymmetric in [0, 2^k - 1]
struct QuantLevels {
  float den, lo, hi;
};
static kt_status quant_levels(const kt_quant_spec* spec, QuantLevels* q) {
  if (!spec) return KT_ERR_INVALID_ARG;
  if (spec->bits < 2 || spec->bits > 8 || (spec->asymmetric != 0 && spec->asymmetric != 1) ||
      !(spec->clip > 0.f && spec->clip <= 1.f) || (spec->clip_mode != 0 && spec->clip_mode != 1) ||
      (spec->clip_mode == 1 && spec->asymmetric != 0))
    return KT_ERR_INVALID_ARG;
  if (spec->asymmetric) {
    q->den = static_cast<float>((1 << spec->bits) - 1);
    q->lo = 0.f;
    q->hi = q->den;
  } else {
    q->den = static_cast<float>((1 << (spec->bits - 1)) - 1);
    q->lo = -q->den;
    q->hi = q->den;
  }
  return KT_OK;
}

// clip_mode 1: position of the clip-quantile among the d sorted magnitudes of a row, h = clip (d - 1) = k0 + t.
static void quantile_position(const kt_quant_spec* spec, int64_t d, int* k0, float* t) {
  *k0 = -1;
  *t = 0.f;
  if (spec->clip_mode != 1) return;
  const double h = static_cast<double>(spec->clip) * static_cast<double>(d - 1);
  const double fl = floor(h);
  *k0 = static_cast<int>(fl);
  *t = static_cast<float>(h - fl);
}

kt_status kt_quant_error(kt_ctx* ctx, kt_mat X, const float* R, const kt_quant_spec* spec, double* mse) {
  if (!ctx || !R || !mse) return KT_ERR_INVALID_ARG;
  QuantLevels q;
  KT_TRY(quant_levels(spec, &q));
  if (spec->clip_mode != 0) return KT_ERR_INVALID_ARG;  // a quantile needs the whole row: kt_quant_error_given
  int64_t N64, d64;
  KT_TRY(check_x(X, &N64, &d64));
  if (!aligned16(R)) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N64, d64, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  const int N = static_cast<int>(N64), d = static_cast<int>(d64);
  XView xv;
  KT_TRY(ingest_x_forward(ctx, X, L, &xv));
  KT_TRY(cast_rt(ctx, R, d, N, L));
  unsigned int* rowmax = at<unsigned int>(ctx, L.rowmax);
  unsigned int* rowmin = spec->asymmetric ? at<unsigned int>(ctx, L.rowmin) : nullptr;
  KT_CUDA(cudaMemsetAsync(rowmax, 0, static_cast<size_t>(N) * 4, ctx->stream));
  if (rowmin) KT_CUDA(cudaMemsetAsync(rowmin, 0xff, static_cast<size_t>(N) * 4, ctx->stream));
  {
    GemmParams p = blank_params();
    const FwdOperands f = fwd_operands(ctx, xv, d, N, L, &p);
    p.rowmax = rowmax;
    p.rowmin = rowmin;
    KT_TRY(run_gemm<kAbsMax>(ctx, N, d, d, f.terms, f.A, f.B, p, kCatQuant));
  }
  {
    GemmParams p = blank_params();
    const FwdOperands f = fwd_operands(ctx, xv, d, N, L, &p);
    p.rowmax = rowmax;
    p.rowmin = rowmin;
    p.qerr = at<float>(ctx, L.qerr);
    p.q_clip = spec->clip;
    p.q_den = q.den;
    p.q_lo = q.lo;
    p.q_hi = q.hi;
    KT_TRY(run_gemm<kQuantErr>(ctx, N, d, d, f.terms, f.A, f.B, p, kCatQuant));
  }
  const long long n = static_cast<long long>(L.P) * N;
  k_block_sums_f32<<<1024, 256, 0, ctx->stream>>>(at<float>(ctx, L.qerr), n, at<double>(ctx, L.norm_blocks));
  KT_LAUNCH_CHECK();
  k_final_sum<<<1, 256, 0, ctx->stream>>>(at<double>(ctx, L.norm_blocks), 1024, 1.0 / (static_cast<double>(N) * d),
                                          &ctx->d_blk->sc.qmse, nullptr, nullptr, nullptr);
  KT_LAUNCH_CHECK();
  KT_TRY(sync_scalars(ctx));
  *mse = ctx->h_blk->sc.qmse;
  return isfinite(*mse) ? KT_OK : KT_ERR_NONFINITE;
}

kt_status kt_quant4_error(kt_ctx* ctx, kt_mat X, const float* R, double* mse) {
  kt_quant_spec spec;
  spec.bits = 4;
  spec.asymmetric = 0;
  spec.clip = 1.0f;
  spec.clip_mode = 0;
  return kt_quant_error(ctx, X, R, &spec, mse);
}

kt_status kt_quant_codes(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, const kt_quant_spec* spec, int16_t* codes,
                         float* scales, float* shifts) {
  if (!ctx || !Y || !codes || !scales || !shifts) return KT_ERR_INVALID_ARG;
  QuantLevels q;
  KT_TRY(quant_levels(spec, &q));
  if (N < 1 || d < 1 || N > 0x7fffffffll || d > 0x7fffffffll) return KT_ERR_SHAPE;
  int k0;
  float t;
  quantile_position(spec, d, &k0, &t);
  k_quant_codes<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(Y, static_cast<int>(d), spec->asymmetric,
                                                                   spec->clip, q.den, q.lo, q.hi, codes, scales,
                                                                   shifts, k0, t, nullptr);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

kt_status kt_quant_error_given(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, const kt_quant_spec* spec,
                               double* mse) {
  if (!ctx || !Y || !mse) return KT_ERR_INVALID_ARG;
  QuantLevels q;
  KT_TRY(quant_levels(spec, &q));
  if (N < 1 || d < 1 || N > 0x7fffffffll || d > 0x7fffffffll) return KT_ERR_SHAPE;
  // one double per row, then a fixed-order sum: the workspace must hold N doubles
  if (ctx->ws == nullptr || ctx->ws_bytes < static_cast<size_t>(N) * 8) return KT_ERR_WORKSPACE;
  double* row_err = reinterpret_cast<double*>(ctx->ws);
  int k0;
  float t;
  quantile_position(spec, d, &k0, &t);
  k_quant_codes<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(Y, static_cast<int>(d), spec->asymmetric,
                                                                   spec->clip, q.den, q.lo, q.hi, nullptr, nullptr,
                                                                   nullptr, k0, t, row_err);
  KT_LAUNCH_CHECK();
  k_final_sum<<<1, 256, 0, ctx->stream>>>(row_err, static_cast<int>(N), 1.0 / (static_cast<double>(N) * d),
                                          &ctx->d_blk->sc.qmse, nullptr, nullptr, nullptr);
  KT_LAUNCH_CHECK();
  KT_TRY(sync_scalars(ctx));
  *mse = ctx->h_blk->sc.qmse;
  return isfinite(*mse) ? KT_OK : KT_ERR_NONFINITE;
}

kt_status kt_rowmax_success(kt_ctx* ctx, kt_mat X, const float* R_a, const float* R_b, double* rate) {
  if (!ctx || !R_a || !rate) return KT_ERR_INVALID_ARG;
  int64_t N64, d64;
  KT_TRY(check_x(X, &N64, &d64));
  if (!aligned16(R_a) || (R_b && !aligned16(R_b))) return KT_ERR_ALIGN;
  const WsLayout L = make_layout(N64, d64, X.dtype, &ctx->cfg);
  KT_TRY(check_ws(ctx, L));
  const int N = static_cast<int>(N64), d = static_cast<int>(d64);
  XView xv;
  // (the comparison is per token and does not depend on the token's scale: no RMSNorm factors here)
  KT_TRY(ingest_x_forward(ctx, X, L, &xv, false));
  unsigned int* max_a = at<unsigned int>(ctx, L.rowmax);
  unsigned int* max_b = at<unsigned int>(ctx, L.rowmin);
  const float* Rs[2] = {R_a, R_b};
  unsigned int* outs[2] = {max_a, max_b};
  for (int which = 0; which < 2; ++which) {
    if (Rs[which] == nullptr) {  // the un-rotated rows themselves
      k_row_absmax<__nv_bfloat16><<<N, 256, 0, ctx->stream>>>(xv.xb, xv.ldx, d, outs[which]);
      KT_LAUNCH_CHECK();
      continue;
    }
    KT_TRY(cast_rt(ctx, Rs[which], d, N, L));
    KT_CUDA(cudaMemsetAsync(outs[which], 0, static_cast<size_t>(N) * 4, ctx->stream));
    GemmParams p = blank_params();
    const FwdOperands f = fwd_operands(ctx, xv, d, N, L, &p);
    p.rowmax = outs[which];
    KT_TRY(run_gemm<kAbsMax>(ctx, N, d, d, f.terms, f.A, f.B, p, kCatQuant));
  }
  k_count_less<<<L.loss_blocks, 256, 0, ctx->stream>>>(max_a, max_b, N, at<double>(ctx, L.block_loss));
  KT_LAUNCH_CHECK();
  k_final_sum<<<1, 256, 0, ctx->stream>>>(at<double>(ctx, L.block_loss), L.loss_blocks, 1.0 / N,
                                          &ctx->d_blk->sc.qmse, nullptr, nullptr, nullptr);
  KT_LAUNCH_CHECK();
  KT_TRY(sync_scalars(ctx));
  *rate = ctx->h_blk->sc.qmse;
  return KT_OK;
}

kt_status kt_profile_begin(kt_ctx* ctx) {
  if (!ctx) return KT_ERR_INVALID_ARG;
  if (!ctx->prof_ev) {
    ctx->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfPairs];
    ctx->prof_cat = new (std::nothrow) unsigned char[kProfPairs];
    if (!ctx->prof_ev || !ctx->prof_cat) return KT_ERR_CUDA;
    for (int i = 0; i < 2 * kProfPairs; ++i) KT_CUDA(cudaEventCreate(&ctx->prof_ev[i]));
  }
  ctx->prof_used = 0;
  ctx->launches = 0;
  ctx->prof_on = true;
  return KT_OK;
}

kt_status kt_profile_end(kt_ctx* ctx, kt_profile* out) {
  if (!ctx || !out) return KT_ERR_INVALID_ARG;
  memset(out, 0, sizeof(*out));
  ctx->prof_on = false;
  KT_CUDA(cudaStreamSynchronize(ctx->stream));
  out->launches_total = ctx->launches;
  for (int i = 0; i < ctx->prof_used; ++i) {
    float ms = 0.f;
    KT_CUDA(cudaEventElapsedTime(&ms, ctx->prof_ev[2 * i], ctx->prof_ev[2 * i + 1]));
    const int c = ctx->prof_cat[i];
    out->gemm_launches[c] += 1;
    out->gemm_ms[c] += ms;
  }
  return KT_OK;
}

kt_status kt_quant4_codes(kt_ctx* ctx, const float* Y, int64_t N, int64_t d, int8_t* codes, float* scales) {
  if (!ctx || !Y || !codes || !scales) return KT_ERR_INVALID_ARG;
  if (N < 1 || d < 1 || N > 0x7fffffffll || d > 0x7fffffffll) return KT_ERR_SHAPE;
  k_quant4_codes<<<static_cast<unsigned>(N), 256, 0, ctx->stream>>>(Y, static_cast<int>(d), codes, scales);
  KT_LAUNCH_CHECK();
  return KT_OK;
}

// ------------------------------------------------------------------------
// kt_kurtosis_loss_noalloc: the loss for callers that must not allocate.
//
// Scratch that kt_kurtosis_loss takes from the caller's workspace (the bf16
// copies of R^T, the per-column-tile moment records, the per-row records, the
// block sums) and the scalar block that kt_create() would cudaMalloc live here in
// one fixed array inside the library image.  Every GPU that loads the library
// carries these 8 MiB until the process exits.
// ------------------------------------------------------------------------
#define KT_NOALLOC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_noalloc_scratch[KT_NOALLOC_SCRATCH_BYTES];

namespace {

struct NoAllocDevice {
  bool ready;
  kt_ctx ctx;          // plain host struct; its device pointers point into g_noalloc_scratch
  unsigned char* base; // device address of g_noalloc_scratch on this device
};
NoAllocDevice g_noalloc_dev[64];
std::mutex g_noalloc_mutex;

// One-time set-up for the current device: resolves the DEVICE address of the
// scratch array (its name is only a host-side handle in host code and must not be
// handed to a kernel), and looks up what the launches need.  Allocates nothing.
kt_status noalloc_setup(int dev, NoAllocDevice** out) {
  if (dev < 0 || dev >= 64) return KT_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  NoAllocDevice& nd = g_noalloc_dev[dev];
  if (!nd.ready) {
    int major = 0, sms = 0;
    KT_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    KT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (major != 10) return KT_ERR_ARCH;
    void* ptr = nullptr;
    KT_CUDA(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    if (ptr == nullptr) return KT_ERR_CUDA;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return KT_ERR_CUDA;
    memset(&nd.ctx, 0, sizeof(nd.ctx));
    kt_default_config(&nd.ctx.cfg);
    nd.ctx.device = dev;
    nd.ctx.sm_count = sms;
    nd.ctx.encode = reinterpret_cast<EncodeTiledFn>(fn);
    nd.base = static_cast<unsigned char*>(ptr);
    nd.ctx.d_blk = reinterpret_cast<DeviceBlock*>(nd.base);  // scalar block first
    nd.ctx.ws = nd.base;
    nd.ctx.ws_bytes = KT_NOALLOC_SCRATCH_BYTES;
    nd.ready = true;
  }
  *out = &nd;
  return KT_OK;
}

}  // namespace

kt_status kt_kurtosis_loss_noalloc(kt_mat X, const float* R, double* loss_dev, void* cuda_stream) {
  if (!R || !loss_dev) return KT_ERR_INVALID_ARG;
  int64_t N, d;
  KT_TRY(check_x(X, &N, &d));
  if (X.dtype != KT_BF16) return KT_ERR_INVALID_ARG;  // a float32 X would need an N x d scratch copy
  if (!aligned16(R) || (reinterpret_cast<uintptr_t>(loss_dev) & 7u) != 0) return KT_ERR_ALIGN;
  if (N > KT_NOALLOC_MAX_N || d > KT_NOALLOC_MAX_D) return KT_ERR_TOO_LARGE;
  int dev = 0;
  KT_CUDA(cudaGetDevice(&dev));
  // the built-in array that is used is the current device's: the caller's buffers must live there too
  const void* ptrs[3] = {X.data, R, loss_dev};
  for (const void* ptr : ptrs) {
    cudaPointerAttributes pa;
    if (cudaPointerGetAttributes(&pa, ptr) != cudaSuccess) {
      (void)cudaGetLastError();
      return KT_ERR_INVALID_ARG;
    }
    if ((pa.type != cudaMemoryTypeDevice && pa.type != cudaMemoryTypeManaged) || pa.device != dev)
      return KT_ERR_INVALID_ARG;
  }
  NoAllocDevice* nd = nullptr;
  KT_TRY(noalloc_setup(dev, &nd));

  // carve the array: [scalar block][R^T hi][R^T lo][records ...]; sizes are bounded by the maxima above
  WsLayout L;
  memset(&L, 0, sizeof(L));
  L.bn = (d % 256 == 0) ? 128 : 64;  // columns per moment record: half a GEMM column tile
  L.P = static_cast<int>(d / L.bn);
  L.loss_blocks = static_cast<int>((N + 255) / 256);
  size_t off = align_up(sizeof(DeviceBlock), 256);
  auto take = [&](size_t bytes) {
    size_t o = off;
    off = align_up(off + bytes, 256);
    return o;
  };
  const size_t dd = static_cast<size_t>(d) * d;
  L.rt_hi = take(dd * 2);
  L.rt_lo = take(dd * 2);
  L.partial = take(static_cast<size_t>(L.P) * N * 16);
  L.coef = take(static_cast<size_t>(N) * 16);
  L.moments = take(static_cast<size_t>(N) * 16);
  // at least 256 entries: the fused d = 128 kernel writes one partial per CTA here
  L.block_loss = take(static_cast<size_t>(L.loss_blocks > 256 ? L.loss_blocks : 256) * 8);
  L.block_deg = take(static_cast<size_t>(L.loss_blocks > 256 ? L.loss_blocks : 256) * 4);
  L.total = off;
  if (L.total > KT_NOALLOC_SCRATCH_BYTES) return KT_ERR_TOO_LARGE;

  // the shared host-side descriptor is used by one call at a time
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  kt_ctx* ctx = &nd->ctx;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps whatever the previous call left: clear the one word that must start at zero
  // (the time-out flag is only ever raised by atomicMax); everything else is written before it is read
  KT_CUDA(cudaMemsetAsync(&ctx->d_blk->sc, 0, sizeof(Scalars), ctx->stream));
  XView xv;
  memset(&xv, 0, sizeof(xv));
  xv.xb = static_cast<const __nv_bfloat16*>(X.data);
  xv.ldx = X.ld;
  KT_TRY(cast_rt(ctx, R, static_cast<int>(d), N, L));
  // nobody reads the status word of this stream-ordered call on the host: a wait that ran out shows as a NaN loss
  return forward_loss(ctx, xv, static_cast<int>(N), static_cast<int>(d), L, loss_dev, false, true);
}

}  // extern "C"
