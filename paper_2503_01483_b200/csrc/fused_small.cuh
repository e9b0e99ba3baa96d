// Single-pass loss + gradient for d = 128 (one rotation shared by many short rows, e.g. the
// value/KV rotation of Section 3, "Placement of the Rotations").
//
// A whole row of Y = X R fits one 128-column tensor-memory tile, so one CTA can take a tile of 128
// tokens through the complete chain without leaving the SM:
//
//   TMA:  X tile (128 tokens x 128 channels, float16 encoding)        -> shared memory
//   MMA1: C = X Rc (Rc = R with each row's mean taken off, so that C is Y = X R minus its row means;
//             Rc^T resident in shared memory, hi [+ lo])               -> tensor memory
//   epilogue (two groups of 4 warps that take alternate tiles, one row per thread): m2, m4 (Eq. 3),
//             kappa, loss term, then
//             G = a c^3 - ab c as float16 (the gradient w.r.t. C)      -> shared memory
//   MMA2: dRc += X^T G (both operands read token-major straight from the tiles above,
//             "MN-major" shared-memory descriptors)                    -> one persistent accumulator
//
// X is read from HBM exactly once per evaluation; Y and G never leave the SM.  Each CTA ends by
// writing its partial dR (128 x 128 float32) and partial loss; a fixed-order sum over CTAs follows.
//
// What bounds it.  Both products take both operands from shared memory, and such an MMA reads 4 KB + 4 KB per
// 128 x 128 x 16 step of 64 cycles: the whole 128-byte-per-clock port.  Per 32 KB tile of X the kernel moves 192 KB
// through that port (TMA write 32, MMA1 64, G stores 32, MMA2 64), so a tile cannot take fewer than about 1600
// cycles however the stages, warps and buffers are arranged; it takes 1700.  HBM, the tensor pipe and the
// float32 pipes all idle behind that.
//
// Operand encoding.  The kernel does not read the caller's bf16 X but a copy made once per X (k_encode_rows_128):
// every row multiplied by the power of two that brings its largest entry into [1, 2), as float16.  A bf16 value
// has 8 significant bits and float16 holds 11, so the copy is exact (entries more than 2^14 below the row's
// largest one lose bits: less than 2^-25 of the row's size).  Neither the kurtosis of a row nor dL/dR depends on
// the row's scale, so nothing else changes -- except that R can now enter as float16 too, with 2^-12 instead of
// 2^-9 relative rounding at the same tensor-core cost (the systematic error this size is sensitive to, see
// kt_config.forward_terms), that the power sums can never leave float32's range whatever the scale of X, and that
// G fits float16.  The row's mean square (of the encoded row) comes with the copy.
#pragma once
#include <cuda.h>

#include <cuda_fp16.h>

#include "sm100_prims.cuh"

namespace kt {

constexpr int kFsD = 128;          // channels = rows of a token tile
constexpr int kFsThreads = 352;    // warp 0: TMA, warp 1: MMA1, warps 2..5 and 6..9: two epilogue groups, warp 10: MMA2
constexpr int kFsMma2Warp = 10;
constexpr int kFsHalf = 128 * 64 * 2;      // bytes of one 128-row x 64-element swizzled block
constexpr int kFsTile = 2 * kFsHalf;       // one 128 x 128 tile of 16-bit elements
// Shared memory: R^T (hi, and lo when TERMS == 2), four X stages, and the G tiles: one per epilogue group with
// one term, a single one with two.  (Measured with one term: five X stages and a single G tile are 8 % slower
// than four and two, because a group's G stores then wait for MMA2 of the other group's tile.)
template <int TERMS>
struct FusedCfg {
  static constexpr int kStages = 4;
  static constexpr int kGBufs = (TERMS == 1) ? 2 : 1;
  static constexpr int kSmem = 1024 + TERMS * kFsTile /*R^T*/ + kStages * kFsTile + kGBufs * kFsTile /*G*/ + 384;
};

struct FusedParams {
  CUtensorMap tmX;    // encoded X [N][128] float16, box 128 rows x 64
  CUtensorMap tmRhi;  // Rc^T as float16 [128][128], box 128 x 64
  CUtensorMap tmRlo;  // its rounding remainder as float16 (TERMS == 2)
  int N;
  double n_mean;      // tokens the loss is a mean over (N, or all shards' rows in a sharded fit)
  int tiles;          // ceil(N / 128)
  float kappa_t;
  float* dr_partial;        // [gridDim.x][128][128]
  double* loss_partial;     // [gridDim.x]
  unsigned int* deg_partial;// [gridDim.x]
  unsigned int* err_word;
  unsigned long long wait_limit_ns;  // bound of every device-side wait of this launch
  const float* row_ms;      // [N] mean square of every encoded row of X (for the rule that skips rows without spread)
};

// Shared-memory descriptor for an "MN-major" 16-bit operand stored as rows of 64 elements (128 bytes,
// 128-byte swizzle) where the ROW index is the contraction index k and the 64 contiguous elements run
// along M (or N): eight k-rows form a 1024-byte group (stride field), the next 64 elements of M/N live
// `lead_bytes` further on (leading field).
__device__ __forceinline__ uint64_t umma_desc_mnmajor_sw128(uint32_t smem_addr, uint32_t lead_bytes,
                                                            uint32_t stride_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
  d |= static_cast<uint64_t>(lead_bytes >> 4) << 16;
  d |= static_cast<uint64_t>(stride_bytes >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

template <int TERMS>
__global__ void __launch_bounds__(kFsThreads, 1) fused_small_kernel(const __grid_constant__ FusedParams p) {
  constexpr int kGBufs = FusedCfg<TERMS>::kGBufs;
  constexpr int kFsXStages = FusedCfg<TERMS>::kStages;
  // every operand of this kernel is float16 (see the note on the encoding of X at the top of this file)
  constexpr uint32_t kIdescK = umma_idesc_f16_f32(128, 128);                            // both K-major
  constexpr uint32_t kIdescMN = umma_idesc_f16_f32(128, 128) | (1u << 15) | (1u << 16);  // both MN-major
  // tensor memory: Y accumulators at columns 0 (even tiles) and 128 (odd tiles), dR accumulator at 256
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kColDr = 256;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t s_rhi = base;
  const uint32_t s_rlo = base + kFsTile;  // only when TERMS == 2
  const uint32_t s_x = base + TERMS * kFsTile;
  const uint32_t s_g = s_x + kFsXStages * kFsTile;
  const uint32_t bars = s_g + kGBufs * kFsTile;
  auto x_full = [&](int s) { return bars + 8u * s; };
  auto x_empty = [&](int s) { return bars + 8u * (kFsXStages + s); };
  auto y_full = [&](int b) { return bars + 8u * (2 * kFsXStages + b); };
  auto y_empty = [&](int b) { return bars + 8u * (2 * kFsXStages + 2 + b); };
  // one or two G tiles, and in either case two barriers each way (even / odd tiles): with one tile a parity
  // wait then cannot mistake the tile two back for the one it needs
  auto g_full = [&](int b) { return bars + 8u * (2 * kFsXStages + 4 + b); };
  auto g_empty = [&](int b) { return bars + 8u * (2 * kFsXStages + 6 + b); };
  const uint32_t r_full = bars + 8u * (2 * kFsXStages + 8);
  const uint32_t dr_full = bars + 8u * (2 * kFsXStages + 9);
  uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
  // (the barriers take 8 * (2 * kFsXStages + 10) <= 160 bytes)
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gbase + (bars - base) + 160);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  double* sh_loss = reinterpret_cast<double*>(gbase + (bars - base) + 168);             // 8 doubles
  unsigned int* sh_deg = reinterpret_cast<unsigned int*>(gbase + (bars - base) + 232);  // 8 words

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  // tiles of this CTA: blockIdx.x, blockIdx.x + gridDim.x, ...
  const int my_tiles = (p.tiles > static_cast<int>(blockIdx.x))
                           ? (p.tiles - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1
                           : 0;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    prefetch_tensormap(&p.tmX);
    prefetch_tensormap(&p.tmRhi);
    prefetch_tensormap(&p.tmRlo);
  }
  if (warp == 1) {
    if (lane == 0) {
      for (int s = 0; s < kFsXStages; ++s) {
        mbar_init(x_full(s), 1);
        mbar_init(x_empty(s), 1);
      }
      for (int b = 0; b < 2; ++b) {
        mbar_init(y_full(b), 1);
        mbar_init(y_empty(b), 4);
      }
      for (int b = 0; b < 2; ++b) {
        mbar_init(g_full(b), 4);
        mbar_init(g_empty(b), 1);
      }
      mbar_init(r_full, 1);
      mbar_init(dr_full, 1);
      fence_barrier_init();
    }
    __syncwarp();
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && my_tiles > 0) {
      mbar_arrive_expect_tx(r_full, static_cast<uint32_t>(TERMS) * kFsTile);
      tma_load_2d(s_rhi, &p.tmRhi, 0, 0, r_full);
      tma_load_2d(s_rhi + kFsHalf, &p.tmRhi, 64, 0, r_full);
      if (TERMS == 2) {
        tma_load_2d(s_rlo, &p.tmRlo, 0, 0, r_full);
        tma_load_2d(s_rlo + kFsHalf, &p.tmRlo, 64, 0, r_full);
      }
      bool ok = true;
      uint32_t issued = 0, last_parity = 0;
      // (asking for the tiles into L2 ahead of their shared-memory load was measured and costs time: the loads alone
      // already run at 0.85 of the copy bandwidth, and the extra requests only add to the memory system's queues)
      for (int n = 0; n < my_tiles; ++n) {
        const int s = n % kFsXStages;
        const uint32_t ph = (n / kFsXStages) & 1;
        if (!mbar_poll_bounded(x_empty(s), ph ^ 1u, abort_flag, 11u, p.wait_limit_ns)) {
          ok = false;
          break;
        }
        const int row0 = (static_cast<int>(blockIdx.x) + n * static_cast<int>(gridDim.x)) * 128;
        mbar_arrive_expect_tx(x_full(s), kFsTile);
        tma_load_2d(s_x + s * kFsTile, &p.tmX, 0, row0, x_full(s));
        tma_load_2d(s_x + s * kFsTile + kFsHalf, &p.tmX, 64, row0, x_full(s));
        issued |= 1u << s;
        last_parity = (last_parity & ~(1u << s)) | (ph << s);
      }
      if (!ok) {
        // leave no copy in flight behind: wait (bounded) for every load issued
        for (int s = 0; s < kFsXStages; ++s) {
          if (!(issued & (1u << s))) continue;
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(x_full(s), (last_parity >> s) & 1u)) {
            if (global_timer_ns() - t0 > 1000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer, first stream
    // MMA1 stream: Y(n) = X(n) Rc as soon as tile n is in shared memory and its Y accumulator has been read out.
    // (MMA2 has a warp of its own, below: one thread feeding both streams is blocked in the issue of one while the
    // other's barrier completes -- measured: 680 cycles from "G written" to the first MMA2, with the tile's
    // shared-memory stage held all the while.)
    if (lane == 0 && my_tiles > 0) {
      bool ok = mbar_wait_bounded(r_full, 0u, abort_flag, 12u, p.wait_limit_ns);
      for (int n = 0; n < my_tiles && ok; ++n) {
        const int s = n % kFsXStages;
        const int b = n & 1;
        if (!mbar_poll_bounded(y_empty(b), ((n >> 1) & 1) ^ 1u, abort_flag, 13u, p.wait_limit_ns) ||
            !mbar_poll_bounded(x_full(s), (n / kFsXStages) & 1, abort_flag, 13u, p.wait_limit_ns)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const uint32_t acc_y = tmem_base + static_cast<uint32_t>(b * 128);
        uint32_t first = 1;
#pragma unroll
        for (int q = 0; q < TERMS; ++q) {
          const uint32_t rb = (q == 0) ? s_rhi : s_rlo;
#pragma unroll
          for (int kb = 0; kb < 2; ++kb) {
            const uint64_t a_desc = umma_desc_kmajor_sw128(s_x + s * kFsTile + kb * kFsHalf, 1024);
            const uint64_t b_desc = umma_desc_kmajor_sw128(rb + kb * kFsHalf, 1024);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              tc_mma_bf16(acc_y, a_desc + 2u * kk, b_desc + 2u * kk, kIdescK, first ? 0u : 1u);
              first = 0;
            }
          }
        }
        tc_commit(y_full(b));
      }
    }
  } else if (warp == kFsMma2Warp) {
    // -------------------------------------------------------------- MMA issuer, second stream
    // dR += X(m)^T G(m) as soon as the epilogue has written that tile's G: contraction over the tile's 128 tokens,
    // 16 per MMA = two 8-row groups.
    if (lane == 0 && my_tiles > 0) {
      const uint32_t acc_dr = tmem_base + kColDr;
      bool ok = true;
      for (int m = 0; m < my_tiles && ok; ++m) {
        const int s = m % kFsXStages;
        if (!mbar_poll_bounded(g_full(m & 1), (m >> 1) & 1, abort_flag, 14u, p.wait_limit_ns)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t a_desc = umma_desc_mnmajor_sw128(s_x + s * kFsTile + ks * 2048, kFsHalf, 1024);
          const uint64_t b_desc =
              umma_desc_mnmajor_sw128(s_g + (kGBufs == 2 ? (m & 1) * kFsTile : 0) + ks * 2048, kFsHalf, 1024);
          tc_mma_bf16(acc_dr, a_desc, b_desc, kIdescMN, (m > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(x_empty(s));      // the X tile is free once these MMAs have read it
        tc_commit(g_empty(m & 1));  // and so is the G tile
      }
      if (ok) tc_commit(dr_full);
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    // Group 0 (warps 2..5) takes this CTA's even tiles, group 1 (warps 6..9) the odd ones: two tiles are in
    // flight per scheduler, so the latency of one tile's reduction hides behind the other's arithmetic.
    const int lg = warp & 3;            // tensor-memory lane group of this warp
    const int grp = (warp - 2) >> 2;    // = tile parity = Y accumulator = G buffer
    const int trow = lg * 32 + lane;    // token within the tile (and row of dR at the end)
    const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(lg * 32) << 16);
    double loss_acc = 0.0;
    unsigned int deg_acc = 0;
    bool ok = true;
    for (int n = grp; n < my_tiles && ok; n += 2) {
      const uint32_t par = (n >> 1) & 1;
      // (asked for before the wait for the accumulator, so that the load's latency is not on the tile's path)
      const int row = (static_cast<int>(blockIdx.x) + n * static_cast<int>(gridDim.x)) * 128 + trow;
      const float msx = (row < p.N) ? __ldg(p.row_ms + row) : 0.f;
      const bool got = mbar_wait_bounded(y_full(grp), par, abort_flag, 16u, p.wait_limit_ns);
      if (!__all_sync(0xffffffffu, got)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      uint32_t v[4][32];
      tmem_ld_32x32(lane_addr + static_cast<uint32_t>(grp * 128), v[0]);
      tmem_ld_32x32(lane_addr + static_cast<uint32_t>(grp * 128 + 32), v[1]);
      tmem_ld_32x32(lane_addr + static_cast<uint32_t>(grp * 128 + 64), v[2]);
      tmem_ld_32x32(lane_addr + static_cast<uint32_t>(grp * 128 + 96), v[3]);
      tc_wait_ld();
      // the accumulator can be refilled while this tile is being reduced
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(y_empty(grp));

      // Eq. 3 on the row.  The second operand of MMA1 is Rc^T (R with every row's mean taken off), so the row that
      // comes out of tensor memory is already the centred row c = y - mean(y): its second and fourth power sums are
      // the central moments, and the gradient has no term through the mean.  Two-wide arithmetic (packed f32x2
      // mul/add/fma): this epilogue is bound by the float32 pipe, three operations per entry here and three below.
      float s2, s4;
      auto power_sums = [&]() {
        float2 b2 = make_float2(0.f, 0.f), e2 = b2, b4 = b2, e4 = b2;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float2 c0 = make_float2(__uint_as_float(v[c][j]), __uint_as_float(v[c][j + 1]));
            const float2 c1 = make_float2(__uint_as_float(v[c][j + 2]), __uint_as_float(v[c][j + 3]));
            const float2 q0 = __fmul2_rn(c0, c0), q1 = __fmul2_rn(c1, c1);
            b2 = __fadd2_rn(b2, q0);
            e2 = __fadd2_rn(e2, q1);
            b4 = __ffma2_rn(q0, q0, b4);
            e4 = __ffma2_rn(q1, q1, e4);
          }
        }
        b2 = __fadd2_rn(b2, e2);
        b4 = __fadd2_rn(b4, e4);
        s2 = b2.x + b2.y;
        s4 = b4.x + b4.y;
      };
      power_sums();
      // kappa, the loss term and the coefficients of dL/dc = a c^3 - ab c (in float32), up to the constant factor
      // 4 / (tokens * 128), which is applied once to the summed gradient instead of to every entry (that also keeps
      // G inside float16's range: |c| <= 11.3 sigma and sigma >= 0.09 for a row whose largest entry is in [1, 2)).
      // A row without spread is one whose variance is below 1e-6 of its mean square INCLUDING the mean, which the
      // centred row no longer shows: that mean square is the one of the encoded row of X (an orthogonal R keeps it),
      // handed in per row.  A NaN there (a non-finite entry of X) goes into the loss.
      const float m2 = s2 * (1.0f / 128.0f), m4 = s4 * (1.0f / 128.0f);
      const bool degenerate = !(msx > 0.f) || (m2 <= 1e-6f * msx);
      float ca = 0.f, cab = 0.f;
      if (msx != msx || s4 != s4) {
        if (row < p.N) loss_acc += static_cast<double>(__uint_as_float(0x7fc00000u));
      } else if (!degenerate) {
        const float r = __frcp_rn(m2);
        const float kappa = (m4 * r) * r;
        const float diff = kappa - p.kappa_t;
        const float sgn = (diff > 0.f) ? 1.0f : ((diff < 0.f) ? -1.0f : 0.0f);
        ca = (sgn * r) * r;
        cab = ca * (m4 * r);
        if (row < p.N) loss_acc += static_cast<double>(fabsf(diff));
      } else if (row < p.N) {
        ++deg_acc;
      }
      const float2 ca2 = make_float2(ca, ca), ncab2 = make_float2(-cab, -cab);

      // G = a c^3 - ab c as float16, token-major, into the swizzled tile MMA2 reads
      // with one G tile it is free once MMA2 of the previous tile (the other group's) has read it; with two,
      // once MMA2 of this group's previous tile has
      const int gw = (kGBufs == 2) ? n - 2 : n - 1;
      const bool free_g = (gw < 0) || mbar_wait_bounded(g_empty(gw & 1), (gw >> 1) & 1, abort_flag, 17u, p.wait_limit_ns);
      if (!__all_sync(0xffffffffu, free_g)) {
        ok = false;
        break;
      }
      const uint32_t g_row = s_g + (kGBufs == 2 ? static_cast<uint32_t>(grp) * kFsTile : 0u) + static_cast<uint32_t>(trow) * 128u;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int j8 = 0; j8 < 4; ++j8) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 cc = make_float2(__uint_as_float(v[c][j8 * 8 + 2 * e]),
                                          __uint_as_float(v[c][j8 * 8 + 2 * e + 1]));
            const float2 g = __fmul2_rn(cc, __ffma2_rn(__fmul2_rn(ca2, cc), cc, ncab2));
            __half2 h = __floats2half2_rn(g.x, g.y);
            pk[e] = *reinterpret_cast<uint32_t*>(&h);
          }
          const int chunk = c * 4 + j8;  // 16-byte chunk 0..15 of the 256-byte row
          const uint32_t addr = g_row + static_cast<uint32_t>(chunk >> 3) * kFsHalf +
                                (static_cast<uint32_t>((chunk & 7) ^ (trow & 7)) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]),
                       "r"(pk[3])
                       : "memory");
        }
      }
      fence_proxy_async_smem();  // make the generic-proxy stores visible to the tensor core
      __syncwarp();
      if (lane == 0) mbar_arrive(g_full(n & 1));
    }

    // partial loss of this CTA (fixed order: lanes by shuffle tree, then the eight warps)
    {
      double l = loss_acc;
      unsigned int dg = deg_acc;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        l += __shfl_down_sync(0xffffffffu, l, o);
        dg += __shfl_down_sync(0xffffffffu, dg, o);
      }
      if (lane == 0) {
        sh_loss[grp * 4 + lg] = l;
        sh_deg[grp * 4 + lg] = dg;
      }
    }
    // partial dR of this CTA: each warp writes its 32 rows x 64 columns (group 0 the left half)
    float* dst = p.dr_partial + (static_cast<long long>(blockIdx.x) * 128 + trow) * 128 + grp * 64;
    if (my_tiles > 0 && ok) {
      const bool got = mbar_wait_bounded(dr_full, 0u, abort_flag, 18u, p.wait_limit_ns);
      if (__all_sync(0xffffffffu, got)) {
        tc_fence_after_sync();
        uint32_t w[32];
#pragma unroll 1
        for (int c0 = 0; c0 < 64; c0 += 32) {
          tmem_ld_32x32(lane_addr + kColDr + static_cast<uint32_t>(grp * 64 + c0), w);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            reinterpret_cast<float4*>(dst + c0)[j] =
                make_float4(__uint_as_float(w[4 * j]), __uint_as_float(w[4 * j + 1]), __uint_as_float(w[4 * j + 2]),
                            __uint_as_float(w[4 * j + 3]));
          }
        }
      }
    } else if (my_tiles == 0) {
      for (int j = 0; j < 16; ++j) reinterpret_cast<float4*>(dst)[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0) {
    double l = 0.0;
    unsigned int dg = 0;
    for (int i = 0; i < 8; ++i) {
      l += sh_loss[i];
      dg += sh_deg[i];
    }
    p.loss_partial[blockIdx.x] = l;
    p.deg_partial[blockIdx.x] = dg;
    if (*abort_flag != 0 && p.err_word != nullptr) atomicMax(p.err_word, *abort_flag);
  }
}

}  // namespace kt
