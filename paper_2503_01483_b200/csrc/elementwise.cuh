// Memory-bound kernels around the GEMMs: casts and bf16 splits, transposes, the
// per-row moment merge and loss reduction, the skew/step-size/axpy pieces of the
// Cayley step, the orthogonality guard, the 4-bit quantizer and the rotation
// initialisers.  Every reduction is fixed-order (no floating-point atomics), so
// repeated runs are bit-identical.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace kt {

// Device-resident scalars shared by the kernels of one context.
struct Scalars {
  double loss;              // last loss
  double qmse;              // last quantisation MSE
  float alpha;              // step size of the current Cayley step
  float wnorm;              // ||W||_F of the current step
  unsigned int max_e_bits;  // max|R^T R - I| as float bits
  unsigned int gate;        // 1 = the polish runs
  unsigned int err_word;    // != 0: a bounded wait ran out (code of the waiting role)
  unsigned int deg_rows;    // rows skipped by the last loss
  // adaptive Cayley step (written by k_step_size, read by the kernels of the step)
  unsigned int n_terms;     // series terms P_0 .. P_{n_terms-1} are evaluated (the rest are below float32 resolution)
  unsigned int p0_terms;    // bf16 terms of R used for P_0 = W R
  unsigned int gate_guard;  // 1 = this step measures R^T R - I
  float drift;              // bound on the orthogonality error accumulated since the last measurement
  unsigned int adam_k;      // Cayley Adam: steps taken
  unsigned int guards;      // measurements of R^T R - I since the fit began
  double adam_v;            // Cayley Adam: running mean of ||dR||_F^2
  double adam_r;            // Cayley Adam: (1 - beta1^k) sqrt(v / (1 - beta2^k) + eps) of the current step
  float wop;                // size of W as an operator used by the current step's choices
  unsigned int need_op;     // 1 = the Frobenius norm alone would cost this step extra work: estimate ||W||_2
  double wnorm2;            // ||W||_F^2 of the current step
  unsigned int finish_count;  // blocks of k_fused_finish that are done (back to 0 when the kernel ends)
  unsigned int pad_;
};

constexpr float kDegenerateRel = 1e-6f;

// ------------------------------------------------------------ block reduce
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
  return v;
}
// Sum over a 256-thread block in a fixed order; result valid in thread `lin` 0.
__device__ __forceinline__ double block_sum_256(double v, double* sh /*8*/, int lin) {
  v = warp_sum(v);
  if ((lin & 31) == 0) sh[lin >> 5] = v;
  __syncthreads();
  double r = 0.0;
  if (lin == 0) {
#pragma unroll
    for (int i = 0; i < 8; ++i) r += sh[i];
  }
  __syncthreads();
  return r;
}

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// ------------------------------------------------------ casts and transposes
// src float32 rows x cols -> bf16 hi (and lo = bf16(src - hi) when lo != null).
// TRANSPOSE: out[c][r], else out[r][c]; ldo = leading dimension of the outputs.
// grid (cols/32, rows/32), block (32, 8); rows and cols multiples of 32.
template <bool TRANSPOSE>
__global__ void k_split_bf16(const float* __restrict__ src, long long ld, __nv_bfloat16* __restrict__ hi,
                             __nv_bfloat16* __restrict__ lo, long long ldo) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  float x[4];  // four independent loads in flight per thread
#pragma unroll
  for (int q = 0; q < 4; ++q) x[q] = src[static_cast<long long>(r0 + ty + 8 * q) * ld + c0 + tx];
  if (!TRANSPOSE) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      __nv_bfloat16 h, l;
      split_bf16(x[q], h, l);
      const long long o = static_cast<long long>(r0 + ty + 8 * q) * ldo + c0 + tx;
      hi[o] = h;
      if (lo) lo[o] = l;
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) tile[ty + 8 * q][tx] = x[q];
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = ty + 8 * q;
      __nv_bfloat16 h, l;
      split_bf16(tile[tx][c], h, l);
      const long long o = static_cast<long long>(c0 + c) * ldo + r0 + tx;
      hi[o] = h;
      if (lo) lo[o] = l;
    }
  }
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// ------------------------------------------- float16 operands of the forward pass
// With R rounded to bf16 the forward GEMM evaluates the loss and the gradient not at R but at bf16(R), 2^-9
// away in every entry -- which, once R has moved off a bf16-exact start by less than that, is a different point
// altogether: measured at d = 4096 after three steps from the Hadamard start, the gradient is then 2.5e-2 of its norm
// away from the float64 one.  float16 keeps three more bits of R at the same tensor-core rate (3e-3 in that case),
// but both operands of an MMA must have the same type, and X is bf16 data with bf16's exponent range.  So the
// forward GEMMs read a copy of X in which every row is multiplied by the power of two that brings its largest
// entry into [1, 2), as float16: exact for bf16 entries within 2^14 of the row's largest, smaller ones lose bits
// worth < 2^-25 of the row's size.  The epilogues multiply the accumulator rows by the inverse factor again (an exact
// operation), so everything after the product sees Y = X R as before.
//
// src: bf16 rows (N x d, leading dimension ld).  x16: N x d float16.  acc[t] = 2^e_t (the inverse of row t's
// factor), times rms[t] when the RMSNorm factors are given: what the epilogues multiply row t by.
// A row with a NaN or Inf becomes all NaN; an all-zero row stays zero with factor 1.  One block of 256 threads per
// row; the row is read twice (the second time from cache).
__global__ void k_encode_rows_f16(const __nv_bfloat16* __restrict__ src, long long ld, int d, __half* __restrict__ x16,
                                  const float* __restrict__ rms, float* __restrict__ acc) {
  __shared__ float shm[8];
  __shared__ int shb[8];
  const __nv_bfloat16* x = src + static_cast<long long>(blockIdx.x) * ld;
  __half* o = x16 + static_cast<long long>(blockIdx.x) * d;
  float amax = 0.f;
  int bad = 0;
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {   // d is a multiple of 128: whole 16-byte pieces
    const uint4 raw = *reinterpret_cast<const uint4*>(x + j);
    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(p2[e]);
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
      bad |= (!(fabsf(f.x) <= 3.4e38f) || !(fabsf(f.y) <= 3.4e38f)) ? 1 : 0;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    bad |= __shfl_xor_sync(0xffffffffu, bad, off);
  }
  if ((threadIdx.x & 31) == 0) {
    shm[threadIdx.x >> 5] = amax;
    shb[threadIdx.x >> 5] = bad;
  }
  __syncthreads();
  amax = shm[0];
  bad = shb[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) {
    amax = fmaxf(amax, shm[i]);
    bad |= shb[i];
  }
  float scale = 1.0f, inv = 1.0f;
  if (amax > 0.f) {
    int e = static_cast<int>((__float_as_uint(amax) >> 23) & 0xffu) - 127;   // amax in [2^e, 2^(e+1)); subnormal: -127
    e = e < -126 ? -126 : (e > 126 ? 126 : e);
    scale = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);           // 2^-e, e in [-126, 126]
    inv = __uint_as_float(static_cast<uint32_t>(127 + e) << 23);             // 2^e
  }
  if (threadIdx.x == 0) acc[blockIdx.x] = (rms != nullptr ? rms[blockIdx.x] : 1.0f) * inv;
  const float nanv = __uint_as_float(0x7fc00000u);
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(x + j);
    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
    uint4 outv;
    __half2* po = reinterpret_cast<__half2*>(&outv);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(p2[e]);
      po[e] = bad ? __floats2half2_rn(nanv, nanv) : __floats2half2_rn(f.x * scale, f.y * scale);
    }
    *reinterpret_cast<uint4*>(o + j) = outv;
  }
}

// R (d x d float32) -> R^T as float16 (the second operand of those GEMMs).  grid (d/32, d/32), block (32, 8).
__global__ void k_rt_f16(const float* __restrict__ R, int d, __half* __restrict__ rt16) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  float x[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) x[q] = R[static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx];
#pragma unroll
  for (int q = 0; q < 4; ++q) tile[ty + 8 * q][tx] = x[q];
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int c = ty + 8 * q;
    rt16[static_cast<long long>(c0 + c) * d + r0 + tx] = __float2half_rn(tile[tx][c]);
  }
}

// X (N x d, leading dimension ld, T = float or bf16) -> Xt (d x ldt bf16, the
// transpose, columns in [N, 64*ceil(N/64)) zero) and, when xb != null, a dense
// bf16 copy Xb (N x d).  grid (d/64, ceil(N/64)), block (32, 8).
template <typename T>
__global__ void k_prepare_x(const T* __restrict__ X, long long ld, int N, int d, __nv_bfloat16* __restrict__ xt,
                            long long ldt, __nv_bfloat16* __restrict__ xb) {
  __shared__ __nv_bfloat16 tile[64][66];
  const int c0 = blockIdx.x * 64, r0 = blockIdx.y * 64;
  const int tx = threadIdx.x, ty = threadIdx.y;
  for (int r = ty; r < 64; r += 8) {
    const int row = r0 + r;
    __nv_bfloat16 v0 = __float2bfloat16_rn(0.f), v1 = v0;
    if (row < N) {
      const T* s = X + static_cast<long long>(row) * ld + c0 + 2 * tx;
      v0 = __float2bfloat16_rn(to_f32(s[0]));
      v1 = __float2bfloat16_rn(to_f32(s[1]));
      if (xb) {
        __nv_bfloat162 pr;
        pr.x = v0;
        pr.y = v1;
        *reinterpret_cast<__nv_bfloat162*>(xb + static_cast<long long>(row) * d + c0 + 2 * tx) = pr;
      }
    }
    tile[r][2 * tx] = v0;
    tile[r][2 * tx + 1] = v1;
  }
  __syncthreads();
  for (int c = ty; c < 64; c += 8) {
    __nv_bfloat162 pr;
    pr.x = tile[2 * tx][c];
    pr.y = tile[2 * tx + 1][c];
    *reinterpret_cast<__nv_bfloat162*>(xt + static_cast<long long>(c0 + c) * ldt + r0 + 2 * tx) = pr;
  }
}

// The same transpose for a bf16 X with no dense copy asked for, in tiles of 64 tokens x 128 channels with 16-byte
// loads (four in flight per thread).  d a multiple of 128.  grid (d/128, ceil(N/64)), block 256.
// bases != null: row t is not X[t] but row t of the minibatch `ids` gathered from several buffers (see
// k_gather_samples for the numbering), read where it lies.
__global__ void k_transpose_x_bf16(const __nv_bfloat16* __restrict__ X, long long ld, int N, int d,
                                   __nv_bfloat16* __restrict__ xt, long long ldt,
                                   const void* const* __restrict__ bases = nullptr, int samples_per_buf = 0,
                                   int rps = 0, const int* __restrict__ ids = nullptr) {
  __shared__ __nv_bfloat16 tile[64][130];
  const int c0 = blockIdx.x * 128, r0 = blockIdx.y * 64;
  const int rr = threadIdx.x >> 4, cc = (threadIdx.x & 15) * 8;  // 16 rows per pass, 8 channels per thread
  uint4 v[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int row = r0 + rr + 16 * q;
    v[q] = make_uint4(0u, 0u, 0u, 0u);
    if (row < N) {
      const __nv_bfloat16* src;
      if (bases != nullptr) {
        const int b = row / rps, r = row - b * rps;
        const int id = ids[b];
        const int buf = id / samples_per_buf, smp = id - buf * samples_per_buf;
        src = static_cast<const __nv_bfloat16*>(bases[buf]) + (static_cast<long long>(smp) * rps + r) * ld;
      } else {
        src = X + static_cast<long long>(row) * ld;
      }
      v[q] = *reinterpret_cast<const uint4*>(src + c0 + cc);
    }
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    unsigned int* dst = reinterpret_cast<unsigned int*>(&tile[rr + 16 * q][cc]);
    dst[0] = v[q].x;
    dst[1] = v[q].y;
    dst[2] = v[q].z;
    dst[3] = v[q].w;
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll 4
  for (int c = w; c < 128; c += 8) {
    __nv_bfloat162 pr;
    pr.x = tile[2 * lane][c];
    pr.y = tile[2 * lane + 1][c];
    *reinterpret_cast<__nv_bfloat162*>(xt + static_cast<long long>(c0 + c) * ldt + r0 + 2 * lane) = pr;
  }
}

// float32 X (N x d, ld) -> dense bf16 Xb (N x d).  grid ceil(N*d/2/256), block 256.
__global__ void k_cast_x(const float* __restrict__ X, long long ld, long long N, int d,
                         __nv_bfloat16* __restrict__ xb) {
  const long long i2 = (static_cast<long long>(blockIdx.x) * 256 + threadIdx.x) * 2;
  if (i2 >= N * d) return;
  const long long row = i2 / d;
  const int col = static_cast<int>(i2 % d);
  const float* s = X + row * ld + col;
  __nv_bfloat162 pr;
  pr.x = __float2bfloat16_rn(s[0]);
  pr.y = __float2bfloat16_rn(s[1]);
  *reinterpret_cast<__nv_bfloat162*>(xb + i2) = pr;
}

// ------------------------------------------------ moments merge and the loss
// Merges the per-column-tile records {mean_p, S2_p, S3_p, S4_p} (each over bn
// columns, central about mean_p) of every row into the row's mean and central
// moments m2, m3, m4 over all d columns (Eq. 3), then kappa = m4/m2^2, the row's
// loss term |kappa - kappa_t| and the coefficients of dL/dY for the backward:
//   G = a c^3 - ab c - am3,  a = sgn(kappa-kappa_t) 4/(N d m2^2), ab = a m4/m2, am3 = a m3.
// A row with m2 <= 1e-6 * (m2 + mean^2), or all zero, contributes nothing.
// grid ceil(N/256), block 256.
// n_mean: the number of tokens the loss is a mean over (N, or more when these rows are one shard of the batch).
// row_scale != null: the rows were multiplied by it in the GEMM epilogue; the coefficients then carry the factor
// too, so that G is the derivative with respect to the unscaled X R.
__global__ void k_moments_finalize(const float4* __restrict__ partial, int P, int N, int d, int bn, float kappa_t,
                                   float4* __restrict__ moments, float4* __restrict__ coef,
                                   double* __restrict__ block_loss, unsigned int* __restrict__ block_deg,
                                   double n_mean, const float* __restrict__ row_scale) {
  __shared__ double sh[8];
  const int row = blockIdx.x * 256 + threadIdx.x;
  double term = 0.0, deg = 0.0;
  if (row < N) {
    double mu = 0.0;
    for (int p = 0; p < P; ++p) mu += static_cast<double>(partial[static_cast<long long>(p) * N + row].x);
    mu /= P;
    double M2 = 0.0, M3 = 0.0, M4 = 0.0;
    const double n = bn;
    for (int p = 0; p < P; ++p) {
      const float4 r = partial[static_cast<long long>(p) * N + row];
      const double dl = static_cast<double>(r.x) - mu, dl2 = dl * dl;
      M2 += r.y + n * dl2;
      M3 += r.z + 3.0 * dl * r.y + n * dl2 * dl;
      M4 += r.w + 4.0 * dl * r.z + 6.0 * dl2 * r.y + n * dl2 * dl2;
    }
    const double m2 = M2 / d, m3 = M3 / d, m4 = M4 / d;
    const double ms = m2 + mu * mu;
    const bool degenerate = (ms == 0.0) || (m2 <= static_cast<double>(kDegenerateRel) * ms);
    float4 cf = make_float4(static_cast<float>(mu), 0.f, 0.f, 0.f);
    if (!degenerate) {
      const double kappa = m4 / (m2 * m2);
      const double diff = kappa - static_cast<double>(kappa_t);
      term = fabs(diff);
      const double sgn = (diff > 0.0) ? 1.0 : ((diff < 0.0) ? -1.0 : 0.0);
      const double rs = row_scale ? static_cast<double>(row_scale[row]) : 1.0;
      const double a = rs * sgn * 4.0 / (n_mean * d * m2 * m2);
      cf.y = static_cast<float>(a);
      cf.z = static_cast<float>(a * m4 / m2);
      cf.w = static_cast<float>(a * m3);
    } else {
      deg = 1.0;
    }
    if (moments)
      moments[row] = make_float4(static_cast<float>(mu), static_cast<float>(m2), static_cast<float>(m3),
                                 static_cast<float>(m4));
    if (coef) coef[row] = cf;
  }
  const double bl = block_sum_256(term, sh, threadIdx.x);
  const double bd = block_sum_256(deg, sh, threadIdx.x);
  if (threadIdx.x == 0) {
    block_loss[blockIdx.x] = bl;
    block_deg[blockIdx.x] = static_cast<unsigned int>(bd);
  }
}

// ------------------------------------------------ backward from a stored Y
// G^T[j][t] = bf16( a c^3 - ab c - am3 ),  c = Y[t][j] - mu, with the row's coefficients coef[t] = {mu, a, ab, am3}
// (the same expression, in the same float32 operations, as the GEMM epilogue that recomputes Y).
// Y is N x d float32 (dense), G^T is d x ldg bf16.  Tiles of 64 tokens x 64 columns through shared memory so that
// both the reads (along d) and the writes (along tokens) are coalesced.  grid (ceil(N/64), d/64): blocks that run
// together write neighbouring 128-byte pieces of the same rows of G^T.  block 256.
__global__ void k_grad_from_y(const float* __restrict__ Y, const float4* __restrict__ coef, int N, int d,
                              __nv_bfloat16* __restrict__ gt, long long ldg) {
  __shared__ __nv_bfloat16 tile[64][66];
  __shared__ float4 cfs[64];
  const int r0 = blockIdx.x * 64, c0 = blockIdx.y * 64;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;  // ty in 0..3
  float y[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    const int row = r0 + ty + 4 * q;
    y[q] = (row < N) ? Y[static_cast<long long>(row) * d + c0 + tx] : 0.f;
  }
  if (threadIdx.x < 64)
    cfs[threadIdx.x] = (r0 + threadIdx.x < N) ? coef[r0 + threadIdx.x] : make_float4(0.f, 0.f, 0.f, 0.f);
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    const int r = ty + 4 * q;
    const float4 cf = cfs[r];
    const float c = y[q] - cf.x;
    // rows past N: y = 0 and zero coefficients give 0; they are not written anyway
    tile[tx][r] = __float2bfloat16_rn(fmaf(c, fmaf(cf.y * c, c, -cf.z), -cf.w));
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;  // 8 warps, each writes 8 of the 64 output rows
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int c = w + 8 * q;
    const int t = r0 + 2 * lane;
    __nv_bfloat16* dst = gt + static_cast<long long>(c0 + c) * ldg + t;
    if (t + 1 < N) {
      *reinterpret_cast<__nv_bfloat162*>(dst) = *reinterpret_cast<const __nv_bfloat162*>(&tile[c][2 * lane]);
    } else if (t < N) {
      dst[0] = tile[c][2 * lane];
    }
  }
}

// The same from the float16 Y (kt_config.backward_mode 0): Y16[t][j] = float16(Y[t][j] * 2^(140 - e)) with one
// exponent byte e per row and run of `bn` columns, yexp[j / bn][t] (written by the forward GEMM's epilogue).
// Tiles of 128 tokens x 64 columns.  16-byte loads: eight threads read the 64 columns of a row, the block's 256
// threads 32 rows at a time, four such loads in flight per thread.  grid (ceil(N/128), d/64), block 256.
__global__ void k_grad_from_y16(const __half* __restrict__ Y, const unsigned char* __restrict__ yexp, int bn,
                                const float4* __restrict__ coef, int N, int d, __nv_bfloat16* __restrict__ gt,
                                long long ldg) {
  // [column][token]; columns 32..63 are shifted by two words so that the eight column groups a warp writes at once
  // fall into different banks
  __shared__ __nv_bfloat16 tile[64][134];
  const int r0 = blockIdx.x * 128, c0 = blockIdx.y * 64;
  const int seg = threadIdx.x & 7, rr = threadIdx.x >> 3;  // 8 columns at c0 + 8 * seg of rows rr + 32 q
  const unsigned char* ex = yexp + static_cast<long long>(c0 / bn) * N;
  uint4 raw[4];
  float4 cf[4];
  float inv[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int row = r0 + rr + 32 * q;
    const bool in = row < N;
    raw[q] = in ? *reinterpret_cast<const uint4*>(Y + static_cast<long long>(row) * d + c0 + 8 * seg)
                : make_uint4(0u, 0u, 0u, 0u);
    cf[q] = in ? coef[row] : make_float4(0.f, 0.f, 0.f, 0.f);
    // 2^(e - 140), e in [14, 254]
    inv[q] = in ? __uint_as_float((static_cast<unsigned int>(ex[row]) - 13u) << 23) : 0.f;
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint32_t w[4] = {raw[q].x, raw[q].y, raw[q].z, raw[q].w};
    const int tr = rr + 32 * q + 4 * (seg >> 2);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 y2 = __half22float2(*reinterpret_cast<const __half2*>(&w[j]));
      const float ca = y2.x * inv[q] - cf[q].x, cb = y2.y * inv[q] - cf[q].x;
      // rows past N: y = 0 and zero coefficients give 0; they are not written anyway
      tile[8 * seg + 2 * j][tr] = __float2bfloat16_rn(fmaf(ca, fmaf(cf[q].y * ca, ca, -cf[q].z), -cf[q].w));
      tile[8 * seg + 2 * j + 1][tr] = __float2bfloat16_rn(fmaf(cb, fmaf(cf[q].y * cb, cb, -cf[q].z), -cf[q].w));
    }
  }
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;  // 8 warps, each writes 8 of the 64 output rows
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int c = w + 8 * q;
    __nv_bfloat16* dst_row = gt + static_cast<long long>(c0 + c) * ldg;
#pragma unroll
    for (int h = 0; h < 2; ++h) {   // two runs of 64 tokens: 128 contiguous bytes per warp and store
      const int tl = 64 * h + 2 * lane;
      const int t = r0 + tl;
      if (t + 1 < N) {
        *reinterpret_cast<__nv_bfloat162*>(dst_row + t) =
            *reinterpret_cast<const __nv_bfloat162*>(&tile[c][tl + 4 * (c >> 5)]);
      } else if (t < N) {
        dst_row[t] = tile[c][tl + 4 * (c >> 5)];
      }
    }
  }
}

// ------------------------------------------- flattened (whole-layer) kurtosis
// The loss of Section 2 taken literally: one kurtosis over the concatenation of all tokens' entries (N*d values).
// The rows' means and central moments (k_moments_finalize) are merged in two fixed-order passes: the global mean
// first, then the central sums about it with the exact shift formulas, all in float64.
// Stage 1: per-block sums of the row means.  grid ceil(N/256), block 256.
__global__ void k_flat_mean(const float4* __restrict__ moments, int N, double* __restrict__ block_out) {
  __shared__ double sh[8];
  const int row = blockIdx.x * 256 + threadIdx.x;
  const double v = (row < N) ? static_cast<double>(moments[row].x) : 0.0;
  const double b = block_sum_256(v, sh, threadIdx.x);
  if (threadIdx.x == 0) block_out[blockIdx.x] = b;
}

// Stage 2: per-block sums of the rows' second, third and fourth central moments shifted to the global mean *mean.
// grid ceil(N/256), block 256; b2/b3/b4 hold one double per block.
__global__ void k_flat_central(const float4* __restrict__ moments, int N, const double* __restrict__ mean,
                               double* __restrict__ b2, double* __restrict__ b3, double* __restrict__ b4) {
  __shared__ double sh[8];
  const int row = blockIdx.x * 256 + threadIdx.x;
  double s2 = 0.0, s3 = 0.0, s4 = 0.0;
  if (row < N) {
    const float4 m = moments[row];
    const double dl = static_cast<double>(m.x) - *mean, dl2 = dl * dl;
    s2 = m.y + dl2;
    s3 = m.z + 3.0 * dl * m.y + dl2 * dl;
    s4 = m.w + 4.0 * dl * m.z + 6.0 * dl2 * m.y + dl2 * dl2;
  }
  s2 = block_sum_256(s2, sh, threadIdx.x);
  s3 = block_sum_256(s3, sh, threadIdx.x);
  s4 = block_sum_256(s4, sh, threadIdx.x);
  if (threadIdx.x == 0) {
    b2[blockIdx.x] = s2;
    b3[blockIdx.x] = s3;
    b4[blockIdx.x] = s4;
  }
}

// One block of 256 threads: global m2, m3, m4, kappa, the loss |kappa - kappa_t| and the coefficients of
// dL/dY = a c^3 - ab c - am3 with c = Y - mean and a = sgn 4/(N d m2^2) (one kurtosis over n = N d values).
// A layer with (numerically) no variance gives loss 0, zero coefficients and deg_rows = N.
// N: rows the moments are a mean over (all shards' rows when the batch is sharded and b2..b4 hold the reduced sums).
__global__ void k_flat_finalize(const double* __restrict__ b2, const double* __restrict__ b3,
                                const double* __restrict__ b4, int nb, long long N, int d, float kappa_t,
                                const double* __restrict__ mean, Scalars* __restrict__ sc,
                                double* __restrict__ hist_slot, float4* __restrict__ coef_global) {
  __shared__ double sh[8];
  double s2 = 0.0, s3 = 0.0, s4 = 0.0;
  for (int i = threadIdx.x; i < nb; i += 256) {
    s2 += b2[i];
    s3 += b3[i];
    s4 += b4[i];
  }
  s2 = block_sum_256(s2, sh, threadIdx.x);
  s3 = block_sum_256(s3, sh, threadIdx.x);
  s4 = block_sum_256(s4, sh, threadIdx.x);
  if (threadIdx.x == 0) {
    const double mu = *mean;
    const double m2 = s2 / N, m3 = s3 / N, m4 = s4 / N;
    const double ms = m2 + mu * mu;
    float4 cf = make_float4(static_cast<float>(mu), 0.f, 0.f, 0.f);
    double loss = 0.0;
    unsigned int deg = 0u;
    if (ms == 0.0 || m2 <= static_cast<double>(kDegenerateRel) * ms) {
      deg = static_cast<unsigned int>(N > 0xffffffffll ? 0xffffffffll : N);
    } else {
      const double kappa = m4 / (m2 * m2);
      const double diff = kappa - static_cast<double>(kappa_t);
      loss = fabs(diff);
      const double sgn = (diff > 0.0) ? 1.0 : ((diff < 0.0) ? -1.0 : 0.0);
      const double a = sgn * 4.0 / (static_cast<double>(N) * d * m2 * m2);
      cf.y = static_cast<float>(a);
      cf.z = static_cast<float>(a * m4 / m2);
      cf.w = static_cast<float>(a * m3);
    }
    *coef_global = cf;
    sc->loss = loss;
    sc->deg_rows = deg;
    if (hist_slot) *hist_slot = loss;
  }
}

// Every row gets the layer's coefficients (times the row's RMSNorm factor when the rows were scaled by one: G is
// the derivative with respect to the unscaled X R).  grid ceil(N/256), block 256.
__global__ void k_flat_fill(const float4* __restrict__ coef_global, int N, float4* __restrict__ coef,
                            const float* __restrict__ row_scale) {
  const int row = blockIdx.x * 256 + threadIdx.x;
  if (row >= N) return;
  float4 c = *coef_global;
  if (row_scale) {
    const float rs = row_scale[row];
    c.y *= rs;
    c.z *= rs;
    c.w *= rs;
  }
  coef[row] = c;
}

// ------------------------------------------------ minibatch of stored samples
// Gathers one minibatch for a rotation shared by several activation buffers: sample ids[b] (b < batch) lives in
// buffer ids[b] / samples_per_buf at rows (ids[b] % samples_per_buf) * rps .. + rps; its rows are copied (and
// rounded to bf16 when T = float) to rows b * rps .. of the dense bf16 matrix out (batch*rps x d).
// grid batch * rps (one block per row), block 256; d a multiple of 8.
template <typename T>
__global__ void k_gather_samples(const void* const* __restrict__ bases, long long ld, int samples_per_buf, int rps,
                                 const int* __restrict__ ids, int d, __nv_bfloat16* __restrict__ out) {
  const int b = blockIdx.x / rps, r = blockIdx.x - b * rps;
  const int id = ids[b];
  const int buf = id / samples_per_buf, smp = id - buf * samples_per_buf;
  const T* src = static_cast<const T*>(bases[buf]) + (static_cast<long long>(smp) * rps + r) * ld;
  __nv_bfloat16* dst = out + static_cast<long long>(blockIdx.x) * d;
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {
    uint4 o;
    __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
    if (sizeof(T) == 2) {
      o = *reinterpret_cast<const uint4*>(src + j);
    } else {
      const float4 a = *reinterpret_cast<const float4*>(src + j);
      const float4 c = *reinterpret_cast<const float4*>(src + j + 4);
      po[0] = __floats2bfloat162_rn(a.x, a.y);
      po[1] = __floats2bfloat162_rn(a.z, a.w);
      po[2] = __floats2bfloat162_rn(c.x, c.y);
      po[3] = __floats2bfloat162_rn(c.z, c.w);
    }
    *reinterpret_cast<uint4*>(dst + j) = o;
  }
}

// ------------------------------------------------------- RMSNorm of the rows
// Eight consecutive elements of a row as float32 (16-byte loads; the row starts on a 16-byte boundary).
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 f = __bfloat1622float2(pr[e]);
    v[2 * e] = f.x;
    v[2 * e + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// rowscale[t] = 1 / sqrt(mean_j x_t[j]^2 + eps): the factor of the unit-gain RMSNorm that follows the rotation in
// the paper's small network (Section 3, "Learning the Rotations").  An orthogonal R keeps every row's norm, so the
// factor of row t of X R is that of row t of X; the GEMM epilogues apply it to the float32 accumulator, and X
// itself is never rescaled or re-rounded.  A row whose mean square plus eps is zero gets the factor 0.
// Row t is X[t] (bases == null), or, for a rotation shared by several buffers, row t of the minibatch `ids`
// gathered from the buffers (see k_gather_samples for the numbering).  xb != null: the row is also copied, as it
// is but rounded to bf16, to row t of the dense matrix xb (the gathered minibatch; the bf16 form of a float32 X).
// mean_square != 0: rowscale[t] receives mean_j x_t[j]^2 itself instead of the factor (the single-pass d = 128
// kernel's measure of a row's size).
// One block of 256 threads per row; T = float or bf16; d a multiple of 8.
template <typename T>
__global__ void k_row_scale(const T* X, long long ld, int d, float eps, float* __restrict__ rowscale,
                            __nv_bfloat16* xb, const void* const* bases, int samples_per_buf, int rps,
                            const int* ids, int mean_square = 0) {
  __shared__ double sh[8];
  const T* x;
  if (bases != nullptr) {
    const int b = blockIdx.x / rps, r = blockIdx.x - b * rps;
    const int id = ids[b];
    const int buf = id / samples_per_buf, smp = id - buf * samples_per_buf;
    x = static_cast<const T*>(bases[buf]) + (static_cast<long long>(smp) * rps + r) * ld;
  } else {
    x = X + static_cast<long long>(blockIdx.x) * ld;
  }
  __nv_bfloat16* o = xb ? xb + static_cast<long long>(blockIdx.x) * d : nullptr;
  float part = 0.f;  // at most d/256 terms per thread in float32, the 256 partials in float64
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {
    float v[8];
    load8(x + j, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) part = fmaf(v[e], v[e], part);
    if (o) {
      uint4 out;
      __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
      for (int e = 0; e < 4; ++e) po[e] = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
      *reinterpret_cast<uint4*>(o + j) = out;
    }
  }
  const double acc = block_sum_256(static_cast<double>(part), sh, threadIdx.x);
  if (threadIdx.x == 0) {
    const double ms = acc / d + static_cast<double>(eps);
    if (mean_square) rowscale[blockIdx.x] = static_cast<float>(acc / d);
    else rowscale[blockIdx.x] = ms > 0.0 ? static_cast<float>(1.0 / sqrt(ms)) : 0.f;
  }
}

// A minibatch gathered from several bf16 buffers straight into the forward pass's float16 encoding: what
// k_row_scale (gather + RMSNorm factor) followed by k_encode_rows_f16 compute, bit for bit, without the dense bf16
// copy in between.  Row t is read where it lies (numbering as in k_gather_samples), twice (the second time from
// cache).  rowscale != null: receives the RMSNorm factor of row t, and acc[t] includes it; null: no RMSNorm.
// One block of 256 threads per row; d a multiple of 128.
__global__ void k_gather_encode_rows_f16(const void* const* __restrict__ bases, long long ld, int samples_per_buf,
                                         int rps, const int* __restrict__ ids, int d, float eps,
                                         float* __restrict__ rowscale, __half* __restrict__ x16,
                                         float* __restrict__ acc) {
  __shared__ double sh[8];
  __shared__ float shm[8];
  __shared__ int shb[8];
  __shared__ float sh_rms;
  const int b = blockIdx.x / rps, r = blockIdx.x - b * rps;
  const int id = ids[b];
  const int buf = id / samples_per_buf, smp = id - buf * samples_per_buf;
  const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(bases[buf]) + (static_cast<long long>(smp) * rps + r) * ld;
  __half* o = x16 + static_cast<long long>(blockIdx.x) * d;
  float part = 0.f, amax = 0.f;
  int bad = 0;
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {
    float v[8];
    load8(x + j, v);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      part = fmaf(v[e], v[e], part);
      amax = fmaxf(amax, fabsf(v[e]));
      bad |= !(fabsf(v[e]) <= 3.4e38f) ? 1 : 0;
    }
  }
  const double sumsq = block_sum_256(static_cast<double>(part), sh, threadIdx.x);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
    bad |= __shfl_xor_sync(0xffffffffu, bad, off);
  }
  if ((threadIdx.x & 31) == 0) {
    shm[threadIdx.x >> 5] = amax;
    shb[threadIdx.x >> 5] = bad;
  }
  if (threadIdx.x == 0) {
    float f = 1.0f;
    if (rowscale != nullptr) {
      const double ms = sumsq / d + static_cast<double>(eps);
      f = ms > 0.0 ? static_cast<float>(1.0 / sqrt(ms)) : 0.f;
      rowscale[blockIdx.x] = f;
    }
    sh_rms = f;
  }
  __syncthreads();
  amax = shm[0];
  bad = shb[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) {
    amax = fmaxf(amax, shm[i]);
    bad |= shb[i];
  }
  float scale = 1.0f, inv = 1.0f;
  if (amax > 0.f) {
    int e = static_cast<int>((__float_as_uint(amax) >> 23) & 0xffu) - 127;   // amax in [2^e, 2^(e+1)); subnormal: -127
    e = e < -126 ? -126 : (e > 126 ? 126 : e);
    scale = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);           // 2^-e, e in [-126, 126]
    inv = __uint_as_float(static_cast<uint32_t>(127 + e) << 23);             // 2^e
  }
  if (threadIdx.x == 0) acc[blockIdx.x] = sh_rms * inv;
  const float nanv = __uint_as_float(0x7fc00000u);
  for (int j = threadIdx.x * 8; j < d; j += 256 * 8) {
    const uint4 raw = *reinterpret_cast<const uint4*>(x + j);
    const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
    uint4 outv;
    __half2* po = reinterpret_cast<__half2*>(&outv);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(p2[e]);
      po[e] = bad ? __floats2half2_rn(nanv, nanv) : __floats2half2_rn(f.x * scale, f.y * scale);
    }
    *reinterpret_cast<uint4*>(o + j) = outv;
  }
}

// One block: *dst = scale * sum(vals[0..n)) (also to *dst2 when not null);
// *count_dst = sum(counts) when counts != null.
// err_word != null: when *err_word is not zero (a bounded wait of an earlier kernel of this call ran out, so the
// sums are not to be trusted) *dst2 receives NaN instead.
__global__ void k_final_sum(const double* __restrict__ vals, int n, double scale, double* __restrict__ dst,
                            double* __restrict__ dst2, const unsigned int* __restrict__ counts,
                            unsigned int* __restrict__ count_dst, const unsigned int* __restrict__ err_word = nullptr) {
  __shared__ double sh[8];
  double s = 0.0, c = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) {
    s += vals[i];
    if (counts) c += counts[i];
  }
  s = block_sum_256(s, sh, threadIdx.x);
  c = block_sum_256(c, sh, threadIdx.x);
  if (threadIdx.x == 0) {
    *dst = s * scale;
    if (dst2) *dst2 = (err_word != nullptr && *err_word != 0u) ? __longlong_as_double(0x7ff8000000000000ll) : s * scale;
    if (count_dst) *count_dst = static_cast<unsigned int>(c);
  }
}

// Sum of float32 values into per-block doubles (fixed order). block 256.
__global__ void k_block_sums_f32(const float* __restrict__ v, long long n, double* __restrict__ block_out) {
  __shared__ double sh[8];
  double s = 0.0;
  for (long long i = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * 256)
    s += v[i];
  s = block_sum_256(s, sh, threadIdx.x);
  if (threadIdx.x == 0) block_out[blockIdx.x] = s;
}

// out[i] = sum over s of part[s * stride + i], s ascending (fixed order).  n a multiple of 4.
// grid ceil(n/4/256), block 256.
// out_hi != null: also out_hi[i] = bf16(out[i]) (the form the Cayley step's first product reads).
__global__ void k_sum_splits(const float* __restrict__ part, int splits, long long stride, long long n,
                             float* __restrict__ out, __nv_bfloat16* __restrict__ out_hi) {
  const long long i4 = (static_cast<long long>(blockIdx.x) * 256 + threadIdx.x) * 4;
  if (i4 >= n) return;
  float4 acc = *reinterpret_cast<const float4*>(part + i4);
  for (int s = 1; s < splits; ++s) {
    const float4 v = *reinterpret_cast<const float4*>(part + s * stride + i4);
    acc.x += v.x;
    acc.y += v.y;
    acc.z += v.z;
    acc.w += v.w;
  }
  *reinterpret_cast<float4*>(out + i4) = acc;
  if (out_hi != nullptr) {
    __nv_bfloat162 lo2 = __floats2bfloat162_rn(acc.x, acc.y), hi2 = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 pk;
    pk.x = *reinterpret_cast<unsigned int*>(&lo2);
    pk.y = *reinterpret_cast<unsigned int*>(&hi2);
    *reinterpret_cast<uint2*>(out_hi + i4) = pk;
  }
}

// --------------------------------------------------------------- Cayley Adam
// M <- beta1 M + (1 - beta1) dR, m_hi = bf16(M), and per-block sums of dR^2.
// grid (d/32, d/32), block (32, 8).
__global__ void k_adam_moment(float* __restrict__ M, const float* __restrict__ dR, float beta1, int d,
                              __nv_bfloat16* __restrict__ m_hi, double* __restrict__ block_g2) {
  __shared__ double sh[8];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  float mv[4], gv[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const long long o = static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx;
    mv[q] = M[o];
    gv[q] = dR[o];
  }
  double acc = 0.0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const long long o = static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx;
    const float m = fmaf(beta1, mv[q], (1.f - beta1) * gv[q]);
    M[o] = m;
    m_hi[o] = __float2bfloat16_rn(m);
    acc += static_cast<double>(gv[q]) * gv[q];
  }
  const int lin = ty * 32 + tx;
  acc = block_sum_256(acc, sh, lin);
  if (lin == 0) block_g2[blockIdx.y * gridDim.x + blockIdx.x] = acc;
}

// One block of 1024 threads: ||dR||_F^2 in fixed order, then the scalar recurrences of Cayley Adam.
__global__ void k_adam_scalars(const double* __restrict__ block_g2, int n, float beta1, float beta2, float adam_eps,
                               Scalars* __restrict__ sc) {
  __shared__ double sh[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += 1024) s += block_g2[i];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    s = 0.0;
    for (int w = 0; w < 32; ++w) s += sh[w];
    const unsigned int k = sc->adam_k + 1u;
    const double b1 = static_cast<double>(beta1), b2 = static_cast<double>(beta2);
    const double v = b2 * sc->adam_v + (1.0 - b2) * s;
    const double vhat = v / (1.0 - pow(b2, static_cast<double>(k)));
    sc->adam_k = k;
    sc->adam_v = v;
    sc->adam_r = (1.0 - pow(b1, static_cast<double>(k))) * sqrt(vhat + static_cast<double>(adam_eps));
  }
}

// Loads the Cayley Adam state that lives on the host between kt_adam_step calls.
__global__ void k_adam_set(Scalars* sc, double v, unsigned int k) {
  sc->adam_v = v;
  sc->adam_k = k;
}

// ------------------------------------------------------------- Cayley pieces
// W = (A - A^T)/2 (divided by adam->adam_r when `adam` is given) for a d x d float32 A, written as bf16 hi (and lo when asked;
// the rounding is odd, so each bf16 part is exactly skew), plus per-block sums of W^2 (of the float32 W).
// grid (d/32, d/32), block (32, 8).
__global__ void k_skew(const float* __restrict__ A, int d, __nv_bfloat16* __restrict__ w_hi,
                       __nv_bfloat16* __restrict__ w_lo, double* __restrict__ block_norm2,
                       const Scalars* __restrict__ adam) {
  __shared__ float tT[32][33];
  __shared__ double sh[8];
  const int bj = blockIdx.x, bi = blockIdx.y;
  const int tx = threadIdx.x, ty = threadIdx.y;
  // Cayley Adam divides the skew part by r (same float for (i, j) and (j, i): W stays exactly skew)
  const float half_scale = adam ? static_cast<float>(0.5 / adam->adam_r) : 0.5f;
  // eight independent loads per thread: four of tile (bi, bj), four of tile (bj, bi) (to be read transposed)
  float av[4], tv[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    av[q] = A[static_cast<long long>(bi * 32 + ty + 8 * q) * d + bj * 32 + tx];
    tv[q] = A[static_cast<long long>(bj * 32 + ty + 8 * q) * d + bi * 32 + tx];
  }
#pragma unroll
  for (int q = 0; q < 4; ++q) tT[ty + 8 * q][tx] = tv[q];
  __syncthreads();
  double acc = 0.0;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int r = ty + 8 * q;
    const long long o = static_cast<long long>(bi * 32 + r) * d + bj * 32 + tx;
    const float w = half_scale * (av[q] - tT[tx][r]);
    __nv_bfloat16 h, l;
    split_bf16(w, h, l);
    w_hi[o] = h;
    if (w_lo) w_lo[o] = l;
    acc += static_cast<double>(w) * w;
  }
  const int lin = ty * 32 + tx;
  acc = block_sum_256(acc, sh, lin);
  if (lin == 0) block_norm2[blockIdx.y * gridDim.x + blockIdx.x] = acc;
}

// y = W v for the d x d bf16 matrix W (row-major) and a float32 vector v; v == null stands for a fixed vector of
// +-1 entries (a hash of the index), the start of the power iteration below.  One warp per row, 8 rows per block:
// grid d/8, block 256.  d is a multiple of 128 (each lane reads 8 consecutive bf16 = 16 bytes at a time).
__device__ __forceinline__ float start_sign(int j) {
  unsigned int h = static_cast<unsigned int>(j) * 2654435761u;
  h ^= h >> 15;
  h *= 2246822519u;
  return ((h >> 13) & 1u) ? 1.f : -1.f;
}
__global__ void k_skew_matvec(const __nv_bfloat16* __restrict__ W, int d, const float* __restrict__ v,
                              float* __restrict__ y, const Scalars* __restrict__ sc) {
  if (sc->need_op == 0u) return;  // the step's choices are already the cheapest with ||W||_F: no estimate needed
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const __nv_bfloat16* w = W + static_cast<long long>(row) * d;
  float acc0 = 0.f, acc1 = 0.f;
  for (int j = lane * 8; j < d; j += 256) {
    const uint4 raw = *reinterpret_cast<const uint4*>(w + j);
    const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&raw);
    float vv[8];
    if (v) {
      const float4 a = *reinterpret_cast<const float4*>(v + j);
      const float4 b = *reinterpret_cast<const float4*>(v + j + 4);
      vv[0] = a.x; vv[1] = a.y; vv[2] = a.z; vv[3] = a.w;
      vv[4] = b.x; vv[5] = b.y; vv[6] = b.z; vv[7] = b.w;
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) vv[e] = start_sign(j + e);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(pr[e]);
      acc0 = fmaf(f.x, vv[2 * e], acc0);
      acc1 = fmaf(f.y, vv[2 * e + 1], acc1);
    }
  }
  float acc = acc0 + acc1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  if (lane == 0) y[row] = acc;
}

// One block of 1024 threads, before the power iteration: ||W||_F^2 in fixed order, and whether the estimate of
// ||W||_2 can change anything this step.  With x_F = alpha ||W||_F: if already x_F / 2 < 2^-11 (one series term) and
// x_F 2^-9 < 2.5e-6 (one bf16 term of R), the step is as cheap as it gets and the matrix-vector products are skipped
// (the drift bound then uses x_F, which only makes the next measurement come a little sooner).
__global__ void k_w_norm(const double* __restrict__ block_norm2, int n, float lr, float q, float eps, int iters,
                         Scalars* __restrict__ sc) {
  __shared__ double sh[32];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += 1024) s += block_norm2[i];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    s = 0.0;
    for (int w = 0; w < 32; ++w) s += sh[w];
    sc->wnorm2 = s;
    const double nrm = sqrt(s);
    const double cap = 2.0 * static_cast<double>(q) / (nrm + static_cast<double>(eps));
    const double a = (static_cast<double>(lr) < cap) ? static_cast<double>(lr) : cap;
    const double x = a * nrm;
    sc->need_op = ((iters >= 1 && 0.5 * x >= ldexp(1.0, -11)) || x * ldexp(1.0, -9) >= 2.5e-6) ? 1u : 0u;
  }
}

// One block of 1024 threads: ||W||_F, alpha = min(lr, 2q/(||W||_F + eps)), and the decisions that depend on
// x = alpha ||W||_2 (bounded by alpha ||W||_F; estimated by a short power iteration when pv_prev/pv_last are given):
//  * n_terms: term k of the series changes R by at most x (x/2)^k (Frobenius bounds the spectral norm, ||R|| = 1);
//    terms below a quarter unit in the last place of a typical entry (2^-26 / sqrt(d)) are skipped (`gate_terms`),
//    and so are terms below a quarter of the error the first term already carries because W enters it as bf16
//    (x 2^-9): (x/2)^k < 2^-11.  What a dropped term would have done for orthogonality (x^2 per step at most) is
//    in the drift bound below and is repaired by the guard;
//  * p0_terms: P_0 = W R multiplies alpha directly; with R as a single bf16 term its error is x 2^-9, which is
//    accepted while that is below 2.5e-6 (a quarter of the default polish threshold), else hi + lo
//    (`cfg_terms` 1..3 forces a count, 0 = this rule);
//  * gate_guard: guard_mode 1 = measure R^T R - I in this step, 2 = do not, 0 = only when the drift bound, which
//    grows by x^2 + x 2^-9 (or x 2^-17 with two terms) + n_terms 2^-23 per step (truncation of the series; rounding
//    of R in P_0; float32 rounding of the update: half an ulp per entry and series term, all aligned, through
//    E = R^T dR + dR^T R with unit columns), has reached half the polish threshold.  A measuring step also clears the running maximum.
__global__ void k_step_size(const double* __restrict__ block_norm2, int n, float lr, float q, float eps,
                            Scalars* __restrict__ sc, int d, int iters, int cfg_terms, int gate_terms, int guard_mode,
                            float thresh, const float* __restrict__ pv_prev, const float* __restrict__ pv_last) {
  // 1024 threads; fixed-order sums: per-thread strided partial, warp shuffle tree, then the 32 warp sums in order
  __shared__ double sh[32];
  __shared__ double tot[3];
  for (int what = 0; what < 3; ++what) {
    double s = 0.0;
    if (what == 0) {
      for (int i = threadIdx.x; i < n; i += 1024) s += block_norm2[i];  // n == 0: k_w_norm has summed already
    } else if (pv_prev && sc->need_op != 0u) {
      const float* v = (what == 1) ? pv_prev : pv_last;
      for (int i = threadIdx.x; i < d; i += 1024) s += static_cast<double>(v[i]) * v[i];
    }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
      s = 0.0;
      for (int w = 0; w < 32; ++w) s += sh[w];
      tot[what] = s;
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double nrm = sqrt(n > 0 ? tot[0] : sc->wnorm2);
    const double cap = 2.0 * static_cast<double>(q) / (nrm + static_cast<double>(eps));
    const double a = (static_cast<double>(lr) < cap) ? static_cast<double>(lr) : cap;
    sc->alpha = static_cast<float>(a);
    sc->wnorm = static_cast<float>(nrm);
    // The step itself uses ||W||_F (above).  The decisions below only need the size of W as an operator: when the
    // power iteration ran, pv_last = W pv_prev, and ||pv_last|| / ||pv_prev|| <= ||W||_2 is its estimate from
    // below; twice that (the iteration is short), capped by the Frobenius norm, stands in for ||W||_2.
    double wop = nrm;
    if (pv_prev && sc->need_op != 0u && tot[1] > 0.0) {
      const double est = 2.0 * sqrt(tot[2] / tot[1]);
      if (est < wop) wop = est;
    }
    sc->wop = static_cast<float>(wop);
    const double x = a * wop;
    unsigned int nt = 1;
    const double floor_k = ldexp(1.0, -26) / sqrt(static_cast<double>(d));
    double bound = x;
    for (int k = 1; k <= iters; ++k) {
      bound *= 0.5 * x;
      if (gate_terms && (bound < floor_k || bound < x * ldexp(1.0, -11))) break;
      ++nt;
    }
    sc->n_terms = nt;
    const unsigned int p0t =
        cfg_terms > 0 ? static_cast<unsigned int>(cfg_terms) : ((x * ldexp(1.0, -9) >= 2.5e-6) ? 2u : 1u);
    sc->p0_terms = p0t;
    unsigned int gg;
    if (guard_mode == 1) {
      gg = 1u;
    } else if (guard_mode == 2) {
      gg = 0u;
    } else {
      const float drift = sc->drift + static_cast<float>(x * x + x * ldexp(1.0, p0t == 1u ? -9 : -17) +
                                                        nt * ldexp(1.0, -23));
      sc->drift = drift;
      gg = (thresh <= 0.f || drift >= 0.5f * thresh) ? 1u : 0u;
    }
    sc->gate_guard = gg;
    if (gg) {
      sc->max_e_bits = 0u;
      sc->guards += 1u;
    }
  }
}

// Start of a fit: no measurement counted yet.
__global__ void k_fit_begin(Scalars* sc) { sc->guards = 0u; }

// Before a measurement outside a step (kt_orth_error): open the guard's gate and clear its running maximum.
__global__ void k_force_guard(Scalars* sc) {
  sc->gate_guard = 1u;
  sc->max_e_bits = 0u;
}

// One term of the Cayley step written as its Neumann series:
//   R_new = R - alpha * sum_{k=0..s} (-alpha/2)^k P_k,   P_0 = W R,  P_{k+1} = W P_k
// (the partial sums are exactly the iterates Y_k of the fixed-point form Y_0 = R - alpha W R,
// Y_k = R - alpha/2 W (R + Y_{k-1})).  This kernel adds term k in place, R += c_k P with
// c_k = -alpha (-alpha/2)^k.  Terms k >= sc->n_terms do nothing.  A term that is not the last one evaluated writes
// P^T as bf16 (pt_hi) for the next product; the last one writes the bf16 forms of the new R instead: r_hi (as is),
// rt_hi/rt_lo (transposed hi/lo) and, when rt16 != null, the transpose as float16 (the forward pass's second operand
// when it runs on float16 operands).  adam_m != null (given with k = 0 only): also M <- adam_r * P.
// grid (d/32, min(d/32, 32)), block (32, 8); each block walks row tiles.
__global__ void k_series_term(float* __restrict__ R, const float* __restrict__ P, const Scalars* __restrict__ sc,
                              int k, int d, __nv_bfloat16* __restrict__ pt_hi, __nv_bfloat16* __restrict__ r_hi,
                              __nv_bfloat16* __restrict__ rt_hi, __nv_bfloat16* __restrict__ rt_lo,
                              float* __restrict__ adam_m, __half* __restrict__ rt16) {
  const unsigned int n_terms = sc->n_terms;
  if (static_cast<unsigned int>(k) >= n_terms) return;
  const bool last = (static_cast<unsigned int>(k) + 1u == n_terms);
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  const float alpha = sc->alpha;
  float ck = -alpha;
  for (int i = 0; i < k; ++i) ck *= -0.5f * alpha;
  const float adam_r = adam_m ? static_cast<float>(sc->adam_r) : 0.f;
  for (int r0 = blockIdx.y * 32; r0 < d; r0 += gridDim.y * 32) {
    float pv[4], rv[4], rn[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const long long o = static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx;
      pv[q] = P[o];
      rv[q] = R[o];
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int r = ty + 8 * q;
      const long long o = static_cast<long long>(r0 + r) * d + c0 + tx;
      rn[q] = fmaf(ck, pv[q], rv[q]);
      R[o] = rn[q];
      if (adam_m) adam_m[o] = adam_r * pv[q];  // Cayley Adam (k = 0 only): M <- r W R
      tile[r][tx] = last ? rn[q] : pv[q];
      if (last) r_hi[o] = __float2bfloat16_rn(rn[q]);
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = ty + 8 * q;
      const long long o = static_cast<long long>(c0 + c) * d + r0 + tx;
      if (last) {
        __nv_bfloat16 h, l;
        split_bf16(tile[tx][c], h, l);
        rt_hi[o] = h;
        rt_lo[o] = l;
        if (rt16) rt16[o] = __float2half_rn(tile[tx][c]);
      } else {
        pt_hi[o] = __float2bfloat16_rn(tile[tx][c]);
      }
    }
    __syncthreads();
  }
}

// The bf16 forms of R that the step and the guard use: r_hi (as is) and rt_hi/rt_lo (transposed).
// grid (d/32, d/32), block (32, 8).
__global__ void k_split_r(const float* __restrict__ R, int d, __nv_bfloat16* __restrict__ r_hi,
                          __nv_bfloat16* __restrict__ rt_hi, __nv_bfloat16* __restrict__ rt_lo) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int r = ty + 8 * q;
    const long long o = static_cast<long long>(r0 + r) * d + c0 + tx;
    const float v = R[o];
    tile[r][tx] = v;
    r_hi[o] = __float2bfloat16_rn(v);
  }
  __syncthreads();
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int c = ty + 8 * q;
    __nv_bfloat16 h, l;
    split_bf16(tile[tx][c], h, l);
    const long long o = static_cast<long long>(c0 + c) * d + r0 + tx;
    rt_hi[o] = h;
    rt_lo[o] = l;
  }
}

// Column sums of squares of a d x d float32 R, by row slabs of 32:
// colpart[slab][j] = sum over the slab's 32 rows of R[i][j]^2.  Does nothing when the guard's gate is closed.
// grid (d/32, min(d/32, 32)), block (32, 8); each block walks row slabs.
__global__ void k_colnorm_partial(const float* __restrict__ R, int d, float* __restrict__ colpart,
                                  const Scalars* __restrict__ sc) {
  if (sc->gate_guard == 0u) return;
  __shared__ float sh[8][33];
  const int c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  for (int slab = blockIdx.y; slab * 32 < d; slab += gridDim.y) {
    const int r0 = slab * 32;
    float v[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) v[q] = R[static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx];
    float acc = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) acc = fmaf(v[q], v[q], acc);
    sh[ty][tx] = acc;
    __syncthreads();
    if (ty == 0) {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) s += sh[i][tx];
      colpart[static_cast<long long>(slab) * d + c0 + tx] = s;
    }
    __syncthreads();
  }
}

// diag[j] = (sum over slabs of colpart[slab][j]) - 1, accumulated in double: the exact diagonal of
// R^T R - I.  One warp per column; grid ceil(d/8), block 256.
__global__ void k_colnorm_final(const float* __restrict__ colpart, int nslabs, int d, float* __restrict__ diag,
                                const Scalars* __restrict__ sc) {
  if (sc->gate_guard == 0u) return;
  const int j = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (j >= d) return;
  double s = 0.0;
  for (int b = threadIdx.x & 31; b < nslabs; b += 32) s += static_cast<double>(colpart[static_cast<long long>(b) * d + j]);
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) diag[j] = static_cast<float>(s - 1.0);
}

// E = S - I for S = R^T R from the tensor cores (d x d float32, of which only the tiles that reach
// the diagonal or lie above it were computed: tile rows of 128, tile columns of bn; the rest is
// taken from the mirror entry).  max|E| goes into sc->max_e_bits (atomic max on the bit pattern of
// a non-negative float: exact, order independent) and E as bf16 into e_hi when not null.
// The diagonal is NOT taken from S: the tensor-core accumulator truncates, which biases a sum of d
// positive terms near 1 by about one unit in the last place per MMA step; `diag` holds it exactly.
// Off-diagonal sums hover around 0 and carry no such bias.  grid (d/32, d/32), block (32, 8).
__global__ void k_guard(const float* __restrict__ S, int d, int bn, const float* __restrict__ diag,
                        __nv_bfloat16* __restrict__ e_hi, Scalars* __restrict__ sc) {
  if (sc->gate_guard == 0u) return;
  __shared__ float tile[32][33];
  __shared__ float shm[8];
  const int c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  float mx = 0.f;
  bool bad = false;
  for (int r0 = blockIdx.y * 32; r0 < d; r0 += gridDim.y * 32) {
    const bool computed = ((c0 / bn) + 1) * bn > (r0 / 128) * 128;
    float e[4];
    if (computed) {
#pragma unroll
      for (int q = 0; q < 4; ++q) e[q] = S[static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx];
    } else {
      float t[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) t[q] = S[static_cast<long long>(c0 + ty + 8 * q) * d + r0 + tx];
#pragma unroll
      for (int q = 0; q < 4; ++q) tile[ty + 8 * q][tx] = t[q];
      __syncthreads();
#pragma unroll
      for (int q = 0; q < 4; ++q) e[q] = tile[tx][ty + 8 * q];
      __syncthreads();
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int row = r0 + ty + 8 * q, col = c0 + tx;
      if (row == col) e[q] = diag[row];
      bad |= (e[q] != e[q]);
      mx = fmaxf(mx, fabsf(e[q]));
      if (e_hi) e_hi[static_cast<long long>(row) * d + col] = __float2bfloat16_rn(e[q]);
    }
  }
  if (bad) mx = __uint_as_float(0x7f800000u);  // a NaN in R^T R reads as +inf
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (tx == 0) shm[ty] = mx;
  __syncthreads();
  if (tx == 0 && ty == 0) {
#pragma unroll
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, shm[i]);
    if (mx > 0.f) atomicMax(&sc->max_e_bits, __float_as_uint(mx));
  }
}

// gate = (max|E| > thresh) when this step measured E.
// `polish_at` <= thresh: inside kt_fit's adaptive cadence the polish already runs at a quarter of the threshold, so
// that the drift bound restarts low and the next measurements can be skipped.
__global__ void k_guard_decide(Scalars* sc, float polish_at) {
  if (sc->gate_guard == 0u) {  // nothing was measured in this step: no polish, the last measurement stands
    sc->gate = 0u;
    return;
  }
  const float mx = __uint_as_float(sc->max_e_bits);
  const unsigned int polish = (mx > polish_at) ? 1u : 0u;
  sc->gate = polish;
  sc->drift = polish ? 0.f : mx;  // the drift bound restarts from what was just measured
}

// When the gate is open: R <- R - Q/2 (one Newton-Schulz step, Q = R E) and the bf16 forms of the
// new R (r_hi, rt_hi, rt_lo, and rt16 when given) are rewritten.  grid (d/32, 16), block (32, 8): each block walks the row tiles
// blockIdx.y, blockIdx.y + 16, ... (a small grid, because in most steps the gate is closed and the kernel only
// has to find that out).
__global__ void k_polish_apply(float* __restrict__ R, const float* __restrict__ Q, const Scalars* __restrict__ sc,
                               int d, __nv_bfloat16* __restrict__ r_hi, __nv_bfloat16* __restrict__ rt_hi,
                               __nv_bfloat16* __restrict__ rt_lo, __half* __restrict__ rt16) {
  if (sc->gate == 0u) return;
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;
  for (int r0 = blockIdx.y * 32; r0 < d; r0 += gridDim.y * 32) {
    float rv[4], qv[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const long long o = static_cast<long long>(r0 + ty + 8 * q) * d + c0 + tx;
      rv[q] = R[o];
      qv[q] = Q[o];
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int r = ty + 8 * q;
      const long long o = static_cast<long long>(r0 + r) * d + c0 + tx;
      const float v = fmaf(-0.5f, qv[q], rv[q]);
      R[o] = v;
      tile[r][tx] = v;
      r_hi[o] = __float2bfloat16_rn(v);
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int c = ty + 8 * q;
      __nv_bfloat16 h, l;
      split_bf16(tile[tx][c], h, l);
      const long long o = static_cast<long long>(c0 + c) * d + r0 + tx;
      rt_hi[o] = h;
      rt_lo[o] = l;
      if (rt16) rt16[o] = __float2half_rn(tile[tx][c]);
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------ quantizer
// One block per row of a dense float32 Y (N x d): s = max|Y_t| / 7 (IEEE divide),
// code = clamp(rint(Y / s), -7, 7) (IEEE divide, ties to even); s == 0 -> zeros.
__global__ void k_quant4_codes(const float* __restrict__ Y, int d, int8_t* __restrict__ codes,
                               float* __restrict__ scales) {
  __shared__ float sh[8];
  const long long base = static_cast<long long>(blockIdx.x) * d;
  float mx = 0.f;
  for (int j = threadIdx.x; j < d; j += 256) mx = fmaxf(mx, fabsf(Y[base + j]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = sh[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) mx = fmaxf(mx, sh[i]);
  const float s = __fdiv_rn(mx, 7.0f);
  if (threadIdx.x == 0) scales[blockIdx.x] = s;
  for (int j = threadIdx.x; j < d; j += 256) {
    float qv = 0.f;
    if (s > 0.f) {
      qv = rintf(__fdiv_rn(Y[base + j], s));
      qv = fminf(fmaxf(qv, -7.0f), 7.0f);
    }
    codes[base + j] = static_cast<int8_t>(qv);
  }
}

// The `level`-quantile of the magnitudes of one row (d float32 values), by the whole block (256 threads), exactly:
// with the magnitudes sorted, a[0] <= ... <= a[d-1], the result is a[k0] + t (a[k0 + 1] - a[k0]) in float32, where
// k0 = floor(level (d - 1)) and t = level (d - 1) - k0 are given by the host (Section 4, "Setup": activations are
// "clipped using a quantile of 0.98").  The order statistic is found by a radix select on the magnitudes' bit
// patterns (which order like the values): four passes over the row, each fixing 8 (the last: 7) more bits of a[k0]
// from a 256-bin histogram of the candidates left; a fifth pass counts the entries <= a[k0] and finds the smallest
// larger one, which is a[k0 + 1] unless a[k0] occurs again.  `hist` (256 words) and `sel` (4 words) are shared
// memory.  Every thread returns the same value.
__device__ float row_abs_quantile(const float* __restrict__ y, int d, int k0, float t, unsigned int* hist,
                                  unsigned int* sel) {
  unsigned int prefix = 0u, mask = 0u, rank = static_cast<unsigned int>(k0);
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 23 - 8 * pass < 0 ? 0 : 23 - 8 * pass;   // 23, 15, 7, 0
    const unsigned int width = pass == 3 ? 0x7fu : 0xffu;
    hist[threadIdx.x] = 0u;
    __syncthreads();
    for (int j = threadIdx.x; j < d; j += 256) {
      const unsigned int key = __float_as_uint(y[j]) & 0x7fffffffu;
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & width], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned int cum = 0u, b = 0u;
      for (; b < width; ++b) {           // (the last bin takes whatever is left)
        if (cum + hist[b] > rank) break;
        cum += hist[b];
      }
      sel[0] = b;
      sel[1] = rank - cum;
    }
    __syncthreads();
    prefix |= sel[0] << shift;
    mask |= width << shift;
    rank = sel[1];
    __syncthreads();
  }
  // prefix = bits of a[k0]; a[k0 + 1]
  unsigned int le = 0u, next = 0x7fffffffu;
  for (int j = threadIdx.x; j < d; j += 256) {
    const unsigned int key = __float_as_uint(y[j]) & 0x7fffffffu;
    if (key <= prefix) ++le;
    else next = key < next ? key : next;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    le += __shfl_xor_sync(0xffffffffu, le, o);
    const unsigned int other = __shfl_xor_sync(0xffffffffu, next, o);
    next = other < next ? other : next;
  }
  if ((threadIdx.x & 31) == 0) {
    hist[threadIdx.x >> 5] = le;
    hist[8 + (threadIdx.x >> 5)] = next;
  }
  __syncthreads();
  le = 0u;
  next = 0x7fffffffu;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    le += hist[i];
    next = hist[8 + i] < next ? hist[8 + i] : next;
  }
  __syncthreads();
  const float a0 = __uint_as_float(prefix);
  const float a1 = (le >= static_cast<unsigned int>(k0) + 2u || k0 + 1 >= d) ? a0 : __uint_as_float(next);
  return __fadd_rn(a0, __fmul_rn(t, __fsub_rn(a1, a0)));
}

// The general k-bit quantizer of Section 2 on a dense float32 Y (N x d), one block per row:
//   symmetric:  s = clip * max|Y_t| / (2^(k-1) - 1), b = 0,            codes in [-(2^(k-1) - 1), 2^(k-1) - 1]
//   asymmetric: b = clip * min Y_t, s = (clip * max Y_t - b) / (2^k - 1), codes in [0, 2^k - 1]
//   code = clamp(rint((y - b) / s), lo, hi); s == 0 -> code 0.  All in IEEE float32, ties to even.
// q_k0 >= 0: the symmetric quantizer's range is the quantile a[q_k0] + q_t (a[q_k0 + 1] - a[q_k0]) of the row's
// magnitudes instead of clip * max|Y_t| (see row_abs_quantile); larger entries saturate.
// err != null: instead of writing codes, the row's sum of (y - Q(y))^2 goes to err[row] (float64; Q(y) = code s + b
// formed in float32).
__global__ void k_quant_codes(const float* __restrict__ Y, int d, int asym, float clip, float den, float lo,
                              float hi, short* __restrict__ codes, float* __restrict__ scales,
                              float* __restrict__ shifts, int q_k0, float q_t, double* __restrict__ err) {
  __shared__ float shx[8], shn[8];
  __shared__ unsigned int hist[256], sel[4];
  __shared__ double she[8];
  const long long base = static_cast<long long>(blockIdx.x) * d;
  float mx = asym ? -INFINITY : 0.f, mn = INFINITY;
  for (int j = threadIdx.x; j < d; j += 256) {
    const float y = Y[base + j];
    mx = fmaxf(mx, asym ? y : fabsf(y));
    mn = fminf(mn, y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  if ((threadIdx.x & 31) == 0) {
    shx[threadIdx.x >> 5] = mx;
    shn[threadIdx.x >> 5] = mn;
  }
  __syncthreads();
  mx = shx[0];
  mn = shn[0];
#pragma unroll
  for (int i = 1; i < 8; ++i) {
    mx = fmaxf(mx, shx[i]);
    mn = fminf(mn, shn[i]);
  }
  float b = 0.f, range;
  if (asym) {
    b = __fmul_rn(clip, mn);
    range = __fsub_rn(__fmul_rn(clip, mx), b);
  } else if (q_k0 >= 0) {
    range = row_abs_quantile(Y + base, d, q_k0, q_t, hist, sel);
  } else {
    range = __fmul_rn(clip, mx);
  }
  const float s = __fdiv_rn(range, den);
  if (threadIdx.x == 0 && scales != nullptr) {
    scales[blockIdx.x] = s;
    shifts[blockIdx.x] = b;
  }
  double e2 = 0.0;
  for (int j = threadIdx.x; j < d; j += 256) {
    const float y = Y[base + j];
    float qv = 0.f;
    if (s > 0.f) {
      qv = rintf(__fdiv_rn(__fsub_rn(y, b), s));
      qv = fminf(fmaxf(qv, lo), hi);
    }
    if (err != nullptr) {
      const double df = static_cast<double>(y) - static_cast<double>(__fadd_rn(__fmul_rn(qv, s), b));
      e2 += df * df;
    } else {
      codes[base + j] = static_cast<short>(qv);
    }
  }
  if (err != nullptr) {   // fixed order: lanes by shuffle tree, then the eight warps
    e2 = warp_sum(e2);
    if ((threadIdx.x & 31) == 0) she[threadIdx.x >> 5] = e2;
    __syncthreads();
    if (threadIdx.x == 0) {
      double t = 0.0;
      for (int i = 0; i < 8; ++i) t += she[i];
      err[blockIdx.x] = t;
    }
  }
}

// Row abs-max of X itself (N x d, T = float or bf16), as float bits: the un-rotated baseline of the success rate.
// One block per row.
template <typename T>
__global__ void k_row_absmax(const T* __restrict__ X, long long ld, int d, unsigned int* __restrict__ rowmax) {
  __shared__ float sh[8];
  const T* x = X + static_cast<long long>(blockIdx.x) * ld;
  float mx = 0.f;
  for (int j = threadIdx.x; j < d; j += 256) mx = fmaxf(mx, fabsf(to_f32(x[j])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    mx = sh[0];
    for (int i = 1; i < 8; ++i) mx = fmaxf(mx, sh[i]);
    rowmax[blockIdx.x] = __float_as_uint(mx);
  }
}

// Per block: how many rows have max_a < max_b (both as bits of non-negative floats).  grid ceil(N/256), block 256.
__global__ void k_count_less(const unsigned int* __restrict__ a, const unsigned int* __restrict__ b, int N,
                             double* __restrict__ block_out) {
  __shared__ double sh[8];
  const int row = blockIdx.x * 256 + threadIdx.x;
  const double v = (row < N && a[row] < b[row]) ? 1.0 : 0.0;
  const double s = block_sum_256(v, sh, threadIdx.x);
  if (threadIdx.x == 0) block_out[blockIdx.x] = s;
}

// ---------------------------------------------------------------- initialisers
// kind 0: identity; kind 1: Sylvester Hadamard (-1)^popcount(i&j) * scale.
__global__ void k_init_rotation(float* __restrict__ R, int d, int kind, float scale) {
  const long long idx = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;
  if (idx >= static_cast<long long>(d) * d) return;
  const int i = static_cast<int>(idx / d), j = static_cast<int>(idx % d);
  float v;
  if (kind == 0) {
    v = (i == j) ? 1.0f : 0.0f;
  } else {
    v = (__popc(i & j) & 1) ? -scale : scale;
  }
  R[idx] = v;
}

}  // namespace kt
