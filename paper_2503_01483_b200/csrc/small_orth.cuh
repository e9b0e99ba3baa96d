// Cayley step + orthogonality guard for small d (128..512) in ONE cooperative launch.
//
// For head-sized rotations the d x d products of the step are a few MFLOP each: as separate
// tensor-core launches they are pure launch latency (about twenty kernels per step).  Here 128 CTAs
// each own d/128 rows of every d x d matrix, compute their rows of each product in float32 on the
// CUDA cores, and meet at grid-wide barriers between products.  Same mathematics as the general path
// (Section 3, "Optimization in the Orthogonal Space"; W = (dR R^T - R dR^T)/2, the Cayley iteration as
// its Neumann series, then E = R^T R - I and one Newton-Schulz step when max|E| is above the
// threshold), but every product is exact float32, so no bf16 split is involved.
#pragma once
#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "elementwise.cuh"

namespace kt {

namespace cg = cooperative_groups;

constexpr int kSoGrid = 128;      // CTAs; each owns d / 128 consecutive rows
constexpr int kSoMaxRows = 4;     // d <= 512
constexpr int kSoD128 = 128 * 128;

// What the single-pass d = 128 loss+gradient kernel leaves behind: one partial dR, loss and count of skipped rows
// per CTA.  Summing them (fixed order) is done either by k_fused_finish or, inside kt_fit, by the first phase of
// small_orth_kernel, which has exactly one thread per entry of dR; both use the functions below, so both give the
// same bits.
struct FusedPartials {
  const float* dr_part;           // [parts][128 * 128]
  int parts;                      // <= 256
  const double* loss_part;        // [parts]
  const unsigned int* deg_part;   // [parts]
  double loss_scale;              // 1 / (tokens the loss is a mean over)
  float dr_scale;                 // 4 / (tokens * 128): the constant factor of dL/dc the kernel leaves out
  int correct;                    // 1: add the first-order term <dR, R - bf16(R)> to the loss
  double* rowdot;                 // [128] scratch: that term, row by row
  double* hist_slot;              // receives the loss too when not null
};

// Entry idx of dR: the partials added in ascending order (loads issued 32 at a time, so that their latency is paid
// five times, not once per partial).
__device__ __forceinline__ float sum_dr_parts(const FusedPartials& f, int idx) {
  float acc = 0.f;
  for (int s0 = 0; s0 < f.parts; s0 += 32) {
    float t[32];
#pragma unroll
    for (int u = 0; u < 32; ++u)
      t[u] = (s0 + u < f.parts) ? __ldcg(f.dr_part + static_cast<long long>(s0 + u) * kSoD128 + idx) : 0.f;
#pragma unroll
    for (int u = 0; u < 32; ++u) acc = (s0 + u == 0) ? t[u] : ((s0 + u < f.parts) ? acc + t[u] : acc);
  }
  return acc * f.dr_scale;
}

// The single-pass kernel's copy of X (128 columns): row t times the power of two that brings its largest entry into
// [1, 2), as float16, and ms[t] = the mean square of that encoded row.  bf16 has 8 significant bits, float16 11: the
// copy is exact but for entries more than 2^14 below the row's largest (they lose bits worth < 2^-25 of the row's
// size).  A float32 X is rounded to bf16 first, as everywhere.  An all-zero row stays zero; a row with a NaN or Inf
// becomes all NaN (and so does the loss).  Row t is X[t] (bases == null) or row t of the minibatch `ids` gathered
// from several buffers (see k_gather_samples for the numbering).  Sixteen lanes per row, eight entries per lane;
// grid ceil(N / 16), block 256.
template <typename T>
__global__ void k_encode_rows_128(const T* __restrict__ X, long long ld, int N, __half* __restrict__ x16,
                                  float* __restrict__ ms, const void* const* __restrict__ bases, int samples_per_buf,
                                  int rps, const int* __restrict__ ids) {
  const int row = blockIdx.x * 16 + (threadIdx.x >> 4);
  const int part = threadIdx.x & 15;
  const bool live = row < N;
  float v[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) v[e] = 0.f;
  if (live) {
    const T* x;
    if (bases != nullptr) {
      const int b = row / rps, r = row - b * rps;
      const int id = ids[b];
      const int buf = id / samples_per_buf, smp = id - buf * samples_per_buf;
      x = static_cast<const T*>(bases[buf]) + (static_cast<long long>(smp) * rps + r) * ld;
    } else {
      x = X + static_cast<long long>(row) * ld;
    }
    load8(x + part * 8, v);
    if (sizeof(T) == 4) {
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __bfloat162float(__float2bfloat16_rn(v[e]));
    }
  }
  float amax = 0.f;
  bool bad = false;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    amax = fmaxf(amax, fabsf(v[e]));
    bad |= !(fabsf(v[e]) <= 3.4e38f);   // NaN or Inf
  }
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) {     // within the row's 16 lanes
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    bad |= (__shfl_xor_sync(0xffffffffu, bad ? 1 : 0, o) != 0);
  }
  float scale = 1.0f;
  if (amax > 0.f) {
    int e = static_cast<int>((__float_as_uint(amax) >> 23) & 0xffu) - 127;   // amax in [2^e, 2^(e+1)); subnormal: -127
    e = e < -126 ? -126 : e;
    scale = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);           // 2^-e, e in [-126, 127]
  }
  float acc = 0.f;
  uint4 out;
  __half2* po = reinterpret_cast<__half2*>(&out);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float a = bad ? __uint_as_float(0x7fc00000u) : v[2 * e] * scale;
    const float b = bad ? __uint_as_float(0x7fc00000u) : v[2 * e + 1] * scale;
    po[e] = __floats2half2_rn(a, b);
    const float2 f = __half22float2(po[e]);
    acc = fmaf(f.x, f.x, acc);
    acc = fmaf(f.y, f.y, acc);
  }
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (live) {
    *reinterpret_cast<uint4*>(x16 + static_cast<long long>(row) * 128 + part * 8) = out;
    if (part == 0) ms[row] = acc * (1.0f / 128.0f);
  }
}

// Mean over a block of 128 threads (one row), in a fixed order, returned to every thread.
__device__ __forceinline__ float row_mean_128(float v, double* sh4) {
  const double w = warp_sum(static_cast<double>(v));
  if ((threadIdx.x & 31) == 0) sh4[threadIdx.x >> 5] = w;
  __syncthreads();
  const float m = static_cast<float>((((sh4[0] + sh4[1]) + sh4[2]) + sh4[3]) * (1.0 / 128.0));
  __syncthreads();
  return m;
}

// The single-pass kernel multiplies X not by R but by Rc = R (I - 1 1^T / d), R with the mean of each row taken off:
// every row of X Rc is the row of X R minus its own mean, so the kernel gets the centred row of Eq. 3 straight out of
// the tensor cores and needs neither the mean nor the mean's part of the gradient.  The chain rule through the
// centring is a projection of the result, dL/dR = (dL/dRc) (I - 1 1^T / d): the mean of each row of the raw gradient
// is taken off again (both by the sums below).
//
// First-order correction of a loss that was evaluated at f16(Rc), Rc rounded to float16, instead of Rc:
//   L = f(Rc) = f(f16 Rc) + <df, Rc - f16 Rc> + O(|Rc - f16 Rc|^2),
// df being the raw gradient at f16(Rc) from the same pass.  The remainder Rc - f16(Rc) is exact in float32 and
// about 2^-12 of Rc, so what is neglected is about 2^-24 of the loss's variation over R.  This is one entry's term.
__device__ __forceinline__ double first_order_term(float dr_raw, float rc) {
  return static_cast<double>(dr_raw) * static_cast<double>(rc - __half2float(__float2half_rn(rc)));
}

// float16 forms of one entry of Rc: the rounded value and the remainder (as the bit patterns the operand buffers,
// which are declared as 16-bit words, receive).
__device__ __forceinline__ void split_f16(float rc, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  const __half h = __float2half_rn(rc);
  const __half l = __float2half_rn(rc - __half2float(h));
  hi = *reinterpret_cast<const __nv_bfloat16*>(&h);
  lo = *reinterpret_cast<const __nv_bfloat16*>(&l);
}

// float16 forms of Rc^T (hi, and lo = the rounding remainder) for the single-pass kernel: one block of 128 threads
// per row of R.  grid 128.
__global__ void __launch_bounds__(128) k_center_split_128(const float* __restrict__ R, __nv_bfloat16* __restrict__ rt_hi,
                                                          __nv_bfloat16* __restrict__ rt_lo) {
  __shared__ double sh4[4];
  const int i = blockIdx.x, j = threadIdx.x;
  const float r = R[i * 128 + j];
  const float rc = r - row_mean_128(r, sh4);
  __nv_bfloat16 h, l;
  split_f16(rc, h, l);
  rt_hi[j * 128 + i] = h;
  rt_lo[j * 128 + i] = l;
}

// Sum over a block of 128 threads in a fixed order (shuffle tree, then the four warps in order); valid in thread 0.
__device__ __forceinline__ double row_sum_128(double v, double* sh4) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) sh4[threadIdx.x >> 5] = v;
  __syncthreads();
  double r = 0.0;
  if (threadIdx.x == 0) r = ((sh4[0] + sh4[1]) + sh4[2]) + sh4[3];
  __syncthreads();
  return r;
}

// One block of 128 threads, after every row's term is in f.rowdot: the loss of the pass and the count of skipped
// rows into the scalar block (values staged through shared memory, then added by one thread in index order).
__device__ __forceinline__ void finish_fused_loss(const FusedPartials& f, Scalars* sc, double* shl /*256*/,
                                                  double* shr /*128*/, unsigned int* shd /*256*/) {
  for (int i = threadIdx.x; i < 256; i += 128) {
    shl[i] = i < f.parts ? __ldcg(f.loss_part + i) : 0.0;
    shd[i] = i < f.parts ? __ldcg(f.deg_part + i) : 0u;
  }
  shr[threadIdx.x] = f.correct ? __ldcg(f.rowdot + threadIdx.x) : 0.0;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0, corr = 0.0;
    unsigned int dg = 0;
    for (int i = 0; i < f.parts; ++i) {
      s += shl[i];
      dg += shd[i];
    }
    for (int i = 0; i < 128; ++i) corr += shr[i];
    const double loss = s * f.loss_scale + corr;
    sc->loss = loss;
    sc->deg_rows = dg;
    if (f.hist_slot) *f.hist_slot = loss;
  }
  __syncthreads();
}

// dR, the loss and the skipped-row count from the partials of the single-pass kernel.  grid 128, block 128: one
// thread per entry of dR, one block per row; the block that finishes last adds up the loss.
__global__ void __launch_bounds__(128) k_fused_finish(const FusedPartials f, const float* __restrict__ R,
                                                      float* __restrict__ dR, Scalars* sc) {
  __shared__ double sh4[4];
  __shared__ double shl[256], shr[128];
  __shared__ unsigned int shd[256];
  __shared__ unsigned int is_last;
  const int idx = blockIdx.x * 128 + threadIdx.x;
  const float acc = sum_dr_parts(f, idx);                 // raw gradient with respect to Rc
  const float r = R[idx];
  const float rc = r - row_mean_128(r, sh4);
  dR[idx] = acc - row_mean_128(acc, sh4);                 // projected: the gradient with respect to R
  const double row = row_sum_128(f.correct ? first_order_term(acc, rc) : 0.0, sh4);
  if (threadIdx.x == 0) {
    f.rowdot[blockIdx.x] = row;
    __threadfence();
    is_last = (atomicAdd(&sc->finish_count, 1u) == gridDim.x - 1u) ? 1u : 0u;
  }
  __syncthreads();
  if (is_last == 0u) return;
  __threadfence();
  finish_fused_loss(f, sc, shl, shr, shd);
  if (threadIdx.x == 0) sc->finish_count = 0u;  // ready for the next call
}

struct SmallOrthParams {
  float* R;            // d x d, in/out
  const float* dR;     // d x d
  int d;
  int iters;           // s: series terms 0..s
  int gate_terms;      // 1: series terms that cannot change the float32 R are not evaluated
  // Cayley Adam (adam_m != null): d x d float32 momentum, in/out; v and the step count live in the scalar block.
  // The direction is then W = skew(M R^T) / r with M <- beta1 M + (1 - beta1) dR, and M <- r W R afterwards.
  float* adam_m;
  float beta1, beta2, adam_eps;
  double* g2_part;     // [kSoGrid] per-CTA sums of dR^2
  int run_guard;       // 1: measure R^T R - I, 0: do not, 2: when the device's drift bound reaches thresh / 2
  float lr, q, eps, thresh;
  float polish_at;     // the polish runs when the measured error exceeds this (<= thresh)
  // scratch, all d x d float32 unless noted
  float* Rt;           // R^T (then R_new^T)
  float* Rs;           // copy of R as it was on entry: what the products read, so that R can be updated in place
                       // without waiting for the other CTAs to finish with it
  float* A;            // dR R^T, later E
  float* W;
  float* P0;           // ping
  float* P1;           // pong
  double* norm_part;   // [kSoGrid]
  float* max_part;     // [kSoGrid]
  Scalars* sc;
  __nv_bfloat16* r_hi; // bf16 forms of the new R for the next loss evaluation
  __nv_bfloat16* rt_hi;
  __nv_bfloat16* rt_lo;
  // d == 128 inside kt_fit: dR is not read from p.dR but summed here from the single-pass kernel's partials
  int use_parts;
  FusedPartials fp;
};

// out[r] = sum_k arow[r][k] * B[k][j] for this thread's column j and the CTA's ROWS rows.
// (B may have been written by other CTAs earlier in this launch: it is read with L2-only loads, never through the
// non-coherent path.)
template <int ROWS>
__device__ __forceinline__ void rows_times_matrix(const float (*arow)[512], const float* B, int d, int j,
                                                  float (&out)[ROWS]) {
#pragma unroll
  for (int r = 0; r < ROWS; ++r) out[r] = 0.f;
#pragma unroll 8
  for (int k = 0; k < d; ++k) {
    const float b = __ldcg(B + static_cast<long long>(k) * d + j);
#pragma unroll
    for (int r = 0; r < ROWS; ++r) out[r] = fmaf(arow[r][k], b, out[r]);
  }
}

// The same with the whole of B (d x d) copied into shared memory first (16-byte L2-only loads, many in flight per
// thread) instead of one load per multiply-add: at d = 128 the d dependent-latency loads of the plain version are
// most of a product's time.  Same operations in the same order: the same bits.  Every thread of the block calls it.
template <int ROWS>
__device__ __forceinline__ void rows_times_staged_matrix(const float (*arow)[512], const float* B, int d, int j,
                                                         float (&out)[ROWS], float* bs) {
  const float4* B4 = reinterpret_cast<const float4*>(B);
  float4* bs4 = reinterpret_cast<float4*>(bs);
  const int n4 = d * d / 4;
  __syncthreads();  // the previous product has finished with bs
#pragma unroll 16
  for (int i = threadIdx.x; i < n4; i += blockDim.x) bs4[i] = __ldcg(B4 + i);
  __syncthreads();
#pragma unroll
  for (int r = 0; r < ROWS; ++r) out[r] = 0.f;
#pragma unroll 8
  for (int k = 0; k < d; ++k) {
    const float b = bs[k * d + j];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) out[r] = fmaf(arow[r][k], b, out[r]);
  }
}

// Sum (or maximum) of the kSoGrid per-CTA partials another phase of this launch left in global memory, the same
// bits in every CTA: thread c < kSoGrid loads partial c (one round trip to L2 for the block, not one per partial),
// the warps reduce with the fixed shuffle tree, and the four warp results are combined in order.  Every thread of
// the block calls it (blockDim.x >= kSoGrid) and gets the result.
__device__ __forceinline__ double sum_of_parts(const double* part, double* sh /*4*/) {
  double v = (threadIdx.x < kSoGrid) ? __ldcg(part + threadIdx.x) : 0.0;
  v = warp_sum(v);
  __syncthreads();  // sh is free
  if (threadIdx.x < kSoGrid && (threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  return ((sh[0] + sh[1]) + sh[2]) + sh[3];
}
__device__ __forceinline__ float max_of_parts(const float* part, float* sh /*4*/) {
  float v = (threadIdx.x < kSoGrid) ? __ldcg(part + threadIdx.x) : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (threadIdx.x < kSoGrid && (threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  return fmaxf(fmaxf(sh[0], sh[1]), fmaxf(sh[2], sh[3]));
}

// Dynamic shared memory: d * d floats when d == 128 (the staged products above), none otherwise.
template <int ROWS>
__global__ void __launch_bounds__(512, 1) small_orth_kernel(const SmallOrthParams p) {
  cg::grid_group grid = cg::this_grid();
  extern __shared__ float4 stage4[];
  float* const bs = reinterpret_cast<float*>(stage4);
  __shared__ float arow[ROWS][512];
  __shared__ double shd[16];
  __shared__ float shf[16];
  const int d = p.d;
  const int j = threadIdx.x;               // column owned by this thread (blockDim.x == d)
  const int i0 = blockIdx.x * ROWS;        // first row owned by this CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;

  auto product = [&](const float* B, float (&out)[ROWS]) {   // out[r] = sum_k arow[r][k] B[k][j]
    if (ROWS == 1 && d == 128) rows_times_staged_matrix<ROWS>(arow, B, d, j, out, bs);
    else rows_times_matrix<ROWS>(arow, B, d, j, out);
  };
  auto load_rows = [&](const float* M) {   // arow[r][:] = M[i0 + r][:]
    __syncthreads();
#pragma unroll
    for (int r = 0; r < ROWS; ++r) arow[r][j] = M[static_cast<long long>(i0 + r) * d + j];
    __syncthreads();
  };

  float rcur[ROWS];  // this thread's entries of the rows of R (then of the new R)
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    rcur[r] = p.R[static_cast<long long>(i0 + r) * d + j];
    p.Rt[static_cast<long long>(j) * d + i0 + r] = rcur[r];
    p.Rs[static_cast<long long>(i0 + r) * d + j] = rcur[r];
  }
  const float drift_in = p.sc->drift;  // (written only by the end of an earlier launch)
  const bool adam = p.adam_m != nullptr;
  const unsigned int adam_k_in = p.sc->adam_k;   // (likewise; block 0 writes the new values after the first barrier)
  const double adam_v_in = p.sc->adam_v;
  float dr_own = 0.f;
  if (ROWS == 1 && p.use_parts) {
    // this CTA's row of dR from the single-pass kernel's partials, and its term of the loss correction
    __shared__ double sh4[4];
    const float raw = sum_dr_parts(p.fp, i0 * d + j);     // raw gradient with respect to Rc (see first_order_term)
    const float rc = rcur[0] - row_mean_128(rcur[0], sh4);
    dr_own = raw - row_mean_128(raw, sh4);
    const double row = row_sum_128(p.fp.correct ? first_order_term(raw, rc) : 0.0, sh4);
    if (threadIdx.x == 0) p.fp.rowdot[blockIdx.x] = row;
  }
  // Cayley Adam: this CTA's rows of M <- beta1 M + (1 - beta1) dR, and its part of ||dR||_F^2
  float mrow[ROWS];
  if (adam) {
    double g2 = 0.0;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      const long long o = static_cast<long long>(i0 + r) * d + j;
      const float g = (ROWS == 1 && p.use_parts) ? dr_own : p.dR[o];
      mrow[r] = fmaf(p.beta1, p.adam_m[o], (1.f - p.beta1) * g);
      g2 += static_cast<double>(g) * g;
    }
    g2 = warp_sum(g2);
    if (lane == 0) shd[warp] = g2;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int w = 0; w < nwarps; ++w) t += shd[w];
      p.g2_part[blockIdx.x] = t;
    }
    __syncthreads();
  }
  grid.sync();
  if (ROWS == 1 && p.use_parts && blockIdx.x == 0) {
    __shared__ double shl[256], shr[128];
    __shared__ unsigned int shdg[256];
    finish_fused_loss(p.fp, p.sc, shl, shr, shdg);
  }
  // r = (1 - beta1^k) sqrt(v / (1 - beta2^k) + eps), the same in every CTA
  double adam_r = 1.0;
  if (adam) {
    const double g2 = sum_of_parts(p.g2_part, shd);
    const unsigned int k = adam_k_in + 1u;
    const double b1 = static_cast<double>(p.beta1), b2 = static_cast<double>(p.beta2);
    const double v = b2 * adam_v_in + (1.0 - b2) * g2;
    const double vhat = v / (1.0 - pow(b2, static_cast<double>(k)));
    adam_r = (1.0 - pow(b1, static_cast<double>(k))) * sqrt(vhat + static_cast<double>(p.adam_eps));
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.sc->adam_k = k;
      p.sc->adam_v = v;
      p.sc->adam_r = adam_r;
    }
  }

  // A = dR R^T (Cayley Adam: M R^T):  A[i][j] = sum_k dR[i][k] Rt[k][j]
  float acc[ROWS];
  if (adam) {
    __syncthreads();
#pragma unroll
    for (int r = 0; r < ROWS; ++r) arow[r][j] = mrow[r];
    __syncthreads();
  } else if (ROWS == 1 && p.use_parts) {
    __syncthreads();
    arow[0][j] = dr_own;
    __syncthreads();
  } else {
    load_rows(p.dR);
  }
  product(p.Rt, acc);
#pragma unroll
  for (int r = 0; r < ROWS; ++r) p.A[static_cast<long long>(i0 + r) * d + j] = acc[r];
  grid.sync();

  // W = (A - A^T)/2 and ||W||_F^2 (per-CTA partial, then every CTA sums the partials in the same order)
  {
    // (Cayley Adam divides the skew part by r: the same float for (i, j) and (j, i), so W stays exactly skew)
    const float half_scale = adam ? static_cast<float>(0.5 / adam_r) : 0.5f;
    double n2 = 0.0;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      const float w = half_scale * (acc[r] - p.A[static_cast<long long>(j) * d + i0 + r]);
      p.W[static_cast<long long>(i0 + r) * d + j] = w;
      n2 += static_cast<double>(w) * w;
    }
    n2 = warp_sum(n2);
    if (lane == 0) shd[warp] = n2;
    __syncthreads();
    if (threadIdx.x == 0) {
      double s = 0.0;
      for (int w = 0; w < nwarps; ++w) s += shd[w];
      p.norm_part[blockIdx.x] = s;
    }
  }
  grid.sync();
  float alpha;
  bool do_guard;   // the same in every CTA
  float drift;     // bound on the orthogonality error accumulated since the last measurement
  int n_terms;     // series terms evaluated (the same in every CTA: the grid-wide barriers below depend on it)
  {
    const double s = sum_of_parts(p.norm_part, shd);
    const double nrm = sqrt(s);
    const double cap = 2.0 * static_cast<double>(p.q) / (nrm + static_cast<double>(p.eps));
    const double a = (static_cast<double>(p.lr) < cap) ? static_cast<double>(p.lr) : cap;
    alpha = static_cast<float>(a);
    // run_guard 1: measure R^T R - I in this step; 0: do not; 2: only when the drift bound asks for it.  Every
    // product here is float32, so a step adds the truncation of the series, 2 x (x/2)^(s+1) with x = alpha ||W||_F
    // (the remainder of the Neumann series, twice through E = R^T dR + dR^T R), and float32 rounding of the update.
    const double x = a * nrm;
    // Term k of the series is at most x (x/2)^k in norm; below 2^-26 / sqrt(d), a quarter ulp of a typical entry of
    // R, it cannot change the float32 R and is not evaluated (what it would have done for orthogonality is part
    // of the drift bound: the truncation below is taken at the last evaluated term).
    n_terms = 1;
    {
      const double floor_k = ldexp(1.0, -26) / sqrt(static_cast<double>(d));
      double bound = x;
      for (int k = 1; k <= p.iters; ++k) {
        bound *= 0.5 * x;
        if (p.gate_terms && bound < floor_k) break;
        ++n_terms;
      }
    }
    double trunc = 2.0 * x;
    for (int k = 0; k < n_terms; ++k) trunc *= 0.5 * x;
    drift = drift_in + static_cast<float>(trunc + (n_terms + 1) * ldexp(1.0, -23));
    do_guard = p.run_guard == 1 || (p.run_guard == 2 && (p.thresh <= 0.f || drift >= 0.5f * p.thresh));
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.sc->alpha = alpha;
      p.sc->wnorm = static_cast<float>(nrm);
      p.sc->wop = static_cast<float>(nrm);  // (every product here is float32: the Frobenius norm is all it needs)
      p.sc->n_terms = static_cast<unsigned int>(n_terms);
      p.sc->p0_terms = 0u;
      if (do_guard) p.sc->guards += 1u;
      else p.sc->drift = drift;
    }
  }

  // R_new = R - alpha sum_k (-alpha/2)^k P_k,  P_0 = W R,  P_{k+1} = W P_k
  load_rows(p.W);
  {
    const float* src = p.Rs;
    float* dst = p.P0;
    float ck = -alpha;
    for (int k = 0; k < n_terms; ++k) {
      product(src, acc);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        rcur[r] = fmaf(ck, acc[r], rcur[r]);
        if (k + 1 < n_terms) dst[static_cast<long long>(i0 + r) * d + j] = acc[r];
        // Cayley Adam: the momentum goes back onto the tangent space at R, M <- r W R
        if (adam && k == 0) p.adam_m[static_cast<long long>(i0 + r) * d + j] = static_cast<float>(adam_r) * acc[r];
      }
      ck *= -0.5f * alpha;
      if (k + 1 < n_terms) {
        grid.sync();  // all rows of P_k written
        src = dst;
        dst = (dst == p.P0) ? p.P1 : p.P0;
      }
    }
  }
  // (no CTA reads R or R^T between the first barrier and the guard's: the products above read the copy)
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    p.R[static_cast<long long>(i0 + r) * d + j] = rcur[r];
    p.Rt[static_cast<long long>(j) * d + i0 + r] = rcur[r];
  }

  float max_e = 0.f;
  if (do_guard) {
    grid.sync();
    // E = R^T R - I:  E[i][j] = sum_k Rt[i][k] R[k][j]
    load_rows(p.Rt);
    product(p.R, acc);
    float mx = 0.f;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      if (i0 + r == j) acc[r] -= 1.0f;
      p.A[static_cast<long long>(i0 + r) * d + j] = acc[r];
      const float av = fabsf(acc[r]);
      mx = (acc[r] != acc[r]) ? __uint_as_float(0x7f800000u) : fmaxf(mx, av);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) shf[warp] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < nwarps; ++w) mx = fmaxf(mx, shf[w]);
      p.max_part[blockIdx.x] = mx;
    }
    grid.sync();
    max_e = max_of_parts(p.max_part, shf);
    if (max_e > p.polish_at) {  // same value in every CTA: the branch is grid-uniform
      // R <- R - R E / 2; each CTA reads only its own rows of R and all of E
      load_rows(p.R);
      product(p.A, acc);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        rcur[r] = fmaf(-0.5f, acc[r], rcur[r]);
        p.R[static_cast<long long>(i0 + r) * d + j] = rcur[r];
      }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.sc->max_e_bits = __float_as_uint(max_e);
      p.sc->gate = (max_e > p.polish_at) ? 1u : 0u;
      p.sc->drift = (max_e > p.polish_at) ? 0.f : max_e;  // the bound restarts from what was just measured
    }
  }

  // bf16 forms of the new R for the next evaluation of the loss (for the single-pass d = 128 kernel: of Rc)
  if (ROWS == 1 && p.use_parts) {
    __shared__ double sh4b[4];
    const float rc = rcur[0] - row_mean_128(rcur[0], sh4b);
    __nv_bfloat16 h, l;
    split_f16(rc, h, l);
    p.r_hi[static_cast<long long>(i0) * d + j] = __float2bfloat16_rn(rcur[0]);
    p.rt_hi[static_cast<long long>(j) * d + i0] = h;
    p.rt_lo[static_cast<long long>(j) * d + i0] = l;
  } else {
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      __nv_bfloat16 h, l;
      split_bf16(rcur[r], h, l);
      p.r_hi[static_cast<long long>(i0 + r) * d + j] = h;
      p.rt_hi[static_cast<long long>(j) * d + i0 + r] = h;
      p.rt_lo[static_cast<long long>(j) * d + i0 + r] = l;
    }
  }
}

}  // namespace kt
