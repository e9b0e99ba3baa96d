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
#include <cuda_runtime.h>

#include "elementwise.cuh"

namespace kt {

namespace cg = cooperative_groups;

constexpr int kSoGrid = 128;      // CTAs; each owns d / 128 consecutive rows
constexpr int kSoMaxRows = 4;     // d <= 512

struct SmallOrthParams {
  float* R;            // d x d, in/out
  const float* dR;     // d x d
  int d;
  int iters;           // s: series terms 0..s
  int run_guard;
  float lr, q, eps, thresh;
  // scratch, all d x d float32 unless noted
  float* Rt;           // R^T (then R_new^T)
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

template <int ROWS>
__global__ void __launch_bounds__(512, 1) small_orth_kernel(const SmallOrthParams p) {
  cg::grid_group grid = cg::this_grid();
  __shared__ float arow[ROWS][512];
  __shared__ double shd[16];
  __shared__ float shf[16];
  const int d = p.d;
  const int j = threadIdx.x;               // column owned by this thread (blockDim.x == d)
  const int i0 = blockIdx.x * ROWS;        // first row owned by this CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;

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
  }
  grid.sync();

  // A = dR R^T:  A[i][j] = sum_k dR[i][k] Rt[k][j]
  float acc[ROWS];
  load_rows(p.dR);
  rows_times_matrix<ROWS>(arow, p.Rt, d, j, acc);
#pragma unroll
  for (int r = 0; r < ROWS; ++r) p.A[static_cast<long long>(i0 + r) * d + j] = acc[r];
  grid.sync();

  // W = (A - A^T)/2 and ||W||_F^2 (per-CTA partial, then every CTA sums the partials in the same order)
  {
    double n2 = 0.0;
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
      const float w = 0.5f * (acc[r] - p.A[static_cast<long long>(j) * d + i0 + r]);
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
  {
    double s = 0.0;
    for (int c = 0; c < kSoGrid; ++c) s += p.norm_part[c];
    const double nrm = sqrt(s);
    const double cap = 2.0 * static_cast<double>(p.q) / (nrm + static_cast<double>(p.eps));
    const double a = (static_cast<double>(p.lr) < cap) ? static_cast<double>(p.lr) : cap;
    alpha = static_cast<float>(a);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.sc->alpha = alpha;
      p.sc->wnorm = static_cast<float>(nrm);
      p.sc->wop = static_cast<float>(nrm);  // this path evaluates every term in float32 and decides nothing
      p.sc->n_terms = static_cast<unsigned int>(p.iters + 1);
      p.sc->p0_terms = 0u;
      if (p.run_guard) p.sc->guards += 1u;
    }
  }

  // R_new = R - alpha sum_k (-alpha/2)^k P_k,  P_0 = W R,  P_{k+1} = W P_k
  load_rows(p.W);
  {
    const float* src = p.R;
    float* dst = p.P0;
    float ck = -alpha;
    for (int k = 0; k <= p.iters; ++k) {
      rows_times_matrix<ROWS>(arow, src, d, j, acc);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        rcur[r] = fmaf(ck, acc[r], rcur[r]);
        if (k < p.iters) dst[static_cast<long long>(i0 + r) * d + j] = acc[r];
      }
      ck *= -0.5f * alpha;
      if (k < p.iters) {
        grid.sync();  // all rows of P_k written; (R itself is not read after the first product)
        src = dst;
        dst = (dst == p.P0) ? p.P1 : p.P0;
      }
    }
  }
  grid.sync();  // every CTA has finished reading R
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    p.R[static_cast<long long>(i0 + r) * d + j] = rcur[r];
    p.Rt[static_cast<long long>(j) * d + i0 + r] = rcur[r];
  }

  float max_e = 0.f;
  if (p.run_guard) {
    grid.sync();
    // E = R^T R - I:  E[i][j] = sum_k Rt[i][k] R[k][j]
    load_rows(p.Rt);
    rows_times_matrix<ROWS>(arow, p.R, d, j, acc);
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
    for (int c = 0; c < kSoGrid; ++c) max_e = fmaxf(max_e, p.max_part[c]);
    if (max_e > p.thresh) {  // same value in every CTA: the branch is grid-uniform
      // R <- R - R E / 2; each CTA reads only its own rows of R and all of E
      load_rows(p.R);
      rows_times_matrix<ROWS>(arow, p.A, d, j, acc);
#pragma unroll
      for (int r = 0; r < ROWS; ++r) {
        rcur[r] = fmaf(-0.5f, acc[r], rcur[r]);
        p.R[static_cast<long long>(i0 + r) * d + j] = rcur[r];
      }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
      p.sc->max_e_bits = __float_as_uint(max_e);
      p.sc->gate = (max_e > p.thresh) ? 1u : 0u;
    }
  }

  // bf16 forms of the new R for the next evaluation of the loss
#pragma unroll
  for (int r = 0; r < ROWS; ++r) {
    __nv_bfloat16 h, l;
    split_bf16(rcur[r], h, l);
    p.r_hi[static_cast<long long>(i0 + r) * d + j] = h;
    p.rt_hi[static_cast<long long>(j) * d + i0 + r] = h;
    p.rt_lo[static_cast<long long>(j) * d + i0 + r] = l;
  }
}

}  // namespace kt
