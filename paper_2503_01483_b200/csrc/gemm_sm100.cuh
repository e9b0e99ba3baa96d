// Persistent, warp-specialised tcgen05 GEMM with fused epilogues.
//
//   D[m][n] = sum over terms q, sum over k of  A_q[m][k] * B_q[n][k]
//
// A_q is M x K and B_q is N x K, both bf16 with k contiguous ("K-major"); the
// accumulator is float32 in tensor memory.  One CTA per SM walks the output
// tiles (128 x BN); warp 0 feeds shared memory with TMA, warp 1 issues the MMAs,
// warps 2..9 drain the accumulator (two warps per 32 rows, half the columns each).  Two accumulators alternate, so the epilogue
// of one tile overlaps the MMAs of the next.  What the epilogue does with a
// finished tile is selected by `EPI`:
//
//   kStoreF32  write D as float32
//   kMoments   per row: mean and central power sums of BN/2 columns (Eq. 3 of the
//              paper, one partial record per half column tile); optionally also
//              stores D as float32, or as float16 with a power-of-two factor per half row
//   kGrad      G = a c^3 - ab c - am3, c = D - mu  (derivative of the loss
//              through Eq. 3), written transposed as bf16
//   kAbsMax    per-row max |D| (first pass of the symmetric quantizer)
//   kQuantErr  per-row sum of (D - Q(D))^2 for the 4-bit symmetric quantizer
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>

#include "sm100_prims.cuh"

namespace kt {

constexpr int kBM = 128;           // rows per tile = tensor-memory lanes
#ifndef KT_GROUP_M
#define KT_GROUP_M 16
#endif
constexpr int kGroupM = KT_GROUP_M;  // row tiles per group of the tile order
constexpr int kBK = 64;            // k elements per pipeline stage (one 128-byte swizzle row)
constexpr int kGemmThreads = 320;  // 10 warps: TMA, MMA, 8 epilogue warps (two per tensor-memory lane quarter)
constexpr int kMaxTerms = 3;

enum Epi : int { kStoreF32 = 0, kMoments = 1, kGrad = 2, kAbsMax = 3, kQuantErr = 4 };

struct GemmParams {
  CUtensorMap tmA[kMaxTerms];
  CUtensorMap tmB[kMaxTerms];
  int terms;
  int M, N, K;
  int m_tiles, n_tiles;
  // split-K (kStoreF32 only): the k-blocks of every tile are cut into k_splits runs of kb_per_split blocks (all
  // non-empty); run s writes its partial tile to out + s * split_stride.  k_splits = 1: no split.
  int k_splits, kb_per_split;
  long long split_stride;
  // upper_only != 0 (square symmetric outputs): tiles that lie entirely below the diagonal are skipped
  int upper_only;
  // epilogue operands (which are used depends on EPI)
  float* out;                 // kStoreF32: M x N, leading dimension ldo; kMoments: the same when not null
  long long ldo;
  int out_sector_aligned;     // out, split_stride*4 and ldo*4 are multiples of 32 bytes: 32-byte stores may be used
  float4* partial;            // kMoments: [2 * n_tiles][M] records {mean, S2, S3, S4}, one per half tile of columns
  const float4* coef;         // kGrad: per row {mu, a, ab, am3}
  __nv_bfloat16* gt;          // kGrad: G transposed, [N][ldg]
  long long ldg;
  // kAbsMax (out) / kQuantErr (in).  Symmetric quantizer (rowmin == null): rowmax = per-row max|D| as float bits.
  // Asymmetric (rowmin != null): rowmax / rowmin = per-row max D / min D as order-preserving keys (ordered_key()).
  unsigned int* rowmax;
  unsigned int* rowmin;
  float* qerr;                // kQuantErr: [2 * n_tiles][M] partial squared errors, one per half tile of columns
  // kQuantErr: step = clip * range / q_den with range = max|D| (symmetric) or max - min (asymmetric, shift =
  // clip * min); codes are clamped to [q_lo, q_hi]
  float q_clip, q_den, q_lo, q_hi;
  const unsigned int* gate;   // when not null and *gate < gate_min the kernel does nothing
  unsigned int gate_min;
  const unsigned int* terms_dev;  // when not null, min(terms, *terms_dev) operand pairs are used
  unsigned int* err_word;     // receives the code of a wait that ran out
  unsigned long long wait_limit_ns;  // bound of every device-side wait of this launch
  // when not null: row m of D is multiplied by row_scale[m] before the epilogue sees it (the RMSNorm that follows
  // the rotation in the paper's small network, applied to the float32 accumulator)
  const float* row_scale;
  // kMoments, when not null: D is kept as float16 (for the backward pass) instead of float32.  Every half row of a
  // tile (the BN/2 columns one thread holds) is multiplied by its own power of two 2^(140 - e), chosen from the half
  // row's mean and sum of squares so that no entry can exceed 2^14; e goes to out16_exp[2 * n_tile + half][row].
  __half* out16;
  unsigned char* out16_exp;
  // != 0: the operands are float16, not bf16 (every term; see k_encode_rows_f16)
  int f16_operands;
};

// Unsigned keys that order like the floats they encode (negative floats reversed, positive ones above them).
__device__ __forceinline__ unsigned int ordered_key(float x) {
  const unsigned int b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ordered_value(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// 32 consecutive float32 of one output row (the accumulator chunk a thread holds): 32-byte stores when the
// destination allows it, 16-byte stores otherwise.
__device__ __forceinline__ void store_row32(float* dst, const uint32_t* v, bool sector_aligned) {
  if (sector_aligned) {
#pragma unroll
    for (int j = 0; j < 4; ++j) st_global_v8(dst + 8 * j, v + 8 * j);
  } else {
    float4* d4 = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      d4[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]),
                          __uint_as_float(v[4 * j + 3]));
    }
  }
}

// CTAS = 2: a pair of CTAs works on a 256 x BN tile; each CTA stages its 128 rows of A and BN/2 rows of B.
template <int BN, int CTAS = 1>
struct GemmSmem {
  static constexpr int kBRows = BN / CTAS;  // rows of B this CTA loads per k-block
  static constexpr int kStages = (kBRows == 256) ? 4 : 6;
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = kBRows * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarBytes = 256;
  static constexpr int kTotal = 1024 /*alignment slack*/ + kStages * kStageBytes + kBarBytes;
};

template <int BN, int EPI, int CTAS = 1>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_tn_kernel(const __grid_constant__ GemmParams p) {
  using S = GemmSmem<BN, CTAS>;
  constexpr int kStages = S::kStages;
  constexpr int kTileM = kBM * CTAS;      // rows of an output tile (of the pair's, when CTAS = 2)
  constexpr int kGroup = kGroupM / CTAS;  // row tiles per group of the tile order
  constexpr uint32_t kTmemCols = 2 * BN;  // two accumulators: 256 or 512 columns
  constexpr uint32_t kIdesc = umma_idesc_bf16_f32(kTileM, BN);
  // CTAS = 2 (launched as clusters of two): rank 0 of a pair is the leader: it issues the MMAs for both and owns the
  // barriers that count loads (full) and drained accumulators (acc_empty); both CTAs own stage (empty) and
  // accumulator-ready (acc_full) barriers, which the leader's commits reach in both at once.
  const uint32_t rank = (CTAS == 2) ? cluster_ctarank() : 0u;
  const int first_unit = blockIdx.x / CTAS, unit_step = gridDim.x / CTAS;

  if (p.gate != nullptr && *p.gate < p.gate_min) return;  // uniform over the grid
  const uint32_t idesc = p.f16_operands ? umma_idesc_f16_f32(kTileM, BN) : kIdesc;
  int n_terms = p.terms;
  if (p.terms_dev != nullptr) {
    const int t = static_cast<int>(*p.terms_dev);
    n_terms = t < n_terms ? (t < 1 ? 1 : t) : n_terms;
  }

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t smem_a = smem_base;
  const uint32_t smem_b = smem_base + kStages * S::kABytes;
  const uint32_t bar_base = smem_base + kStages * S::kStageBytes;
  // barrier slots (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2]
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };
  auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };
  uint8_t* generic_base = smem_raw + (smem_base - smem_u32(smem_raw));
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(generic_base + kStages * S::kStageBytes + 192);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int plain_tiles = p.m_tiles * p.n_tiles;
  const int total_tiles = plain_tiles * p.k_splits;  // work units (k-run, tile), k-run major: CTAs that run
                                                     // together walk the same k range and share operands in L2
  const int k_blocks = (p.K + kBK - 1) / kBK;
  // k-block range and MMA/TMA iteration count of work unit u
  // a tile whose last column is left of its first row holds only entries below the diagonal
  // Tile order: row tiles are taken in groups of kGroupM; inside a group the column tile is the slow index.  The
  // CTAs that run together then cover about kGroupM x (CTAs / kGroupM) tiles, so a wave reads kGroupM row panels of
  // A and CTAs/kGroupM column panels of B instead of a few row panels and all of B (which, once B no longer fits
  // in L2, streamed the whole of B from memory for every two or three row tiles).
  auto tile_mn = [&](int tile, int& mt, int& nt) {
    const int per_group = kGroup * p.n_tiles;
    const int g = tile / per_group, r = tile - g * per_group;
    const int rem = p.m_tiles - g * kGroup;
    const int gm = rem < kGroup ? rem : kGroup;
    nt = r / gm;
    mt = g * kGroup + (r - nt * gm);
  };
  auto skipped = [&](int tile) {
    if (p.upper_only == 0) return false;
    int mt, nt;
    tile_mn(tile, mt, nt);
    return (nt + 1) * BN <= mt * kTileM;
  };
  auto unit_kb0 = [&](int u) { return (u / plain_tiles) * p.kb_per_split; };
  auto unit_iters = [&](int u) {
    const int kb0 = (u / plain_tiles) * p.kb_per_split;
    const int kb1 = (kb0 + p.kb_per_split < k_blocks) ? kb0 + p.kb_per_split : k_blocks;
    return (kb1 - kb0) * n_terms;
  };

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int q = 0; q < p.terms; ++q) {
      prefetch_tensormap(&p.tmA[q]);
      prefetch_tensormap(&p.tmB[q]);
    }
  }
  if (warp == 1) {
    if (lane == 0) {
      for (int s = 0; s < kStages; ++s) {
        mbar_init(full_bar(s), 1);
        mbar_init(empty_bar(s), 1);
      }
      for (int b = 0; b < 2; ++b) {
        mbar_init(acc_full_bar(b), 1);
        mbar_init(acc_empty_bar(b), 8 * CTAS);  // every epilogue warp of every CTA of the tile
      }
      fence_barrier_init();
    }
    __syncwarp();
    if constexpr (CTAS == 2) {
      tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      tmem_relinquish();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if constexpr (CTAS == 2) cluster_sync_all();  // the partner's barriers exist before anything reaches them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t issued_mask = 0;  // stages that have had a load issued
      uint32_t last_parity = 0;  // parity of the last load issued, per stage
      bool ok = true;
      for (int unit = first_unit; unit < total_tiles && ok; unit += unit_step) {
        const int tile = unit % plain_tiles;
        if (skipped(tile)) continue;
        int m_tile, n_tile;
        tile_mn(tile, m_tile, n_tile);
        const int m0 = m_tile * kTileM + static_cast<int>(rank) * kBM;         // this CTA's rows of A
        const int n0 = n_tile * BN + static_cast<int>(rank) * S::kBRows;        // this CTA's rows of B
        const int kb0 = unit_kb0(unit);
        const int iters = unit_iters(unit);
        for (int it = 0; it < iters; ++it) {
          const int kbl = it / n_terms;
          const int q = it - kbl * n_terms;
          const int kb = kb0 + kbl;
          if (!mbar_wait_bounded(empty_bar(stage), phase ^ 1u, abort_flag, 1u, p.wait_limit_ns)) {
            ok = false;
            break;
          }
          if constexpr (CTAS == 2) {
            // both CTAs' bytes are counted on the leader's barrier; only the leader announces them
            if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * S::kStageBytes);
            const uint32_t lead_full = cluster_map_shared(full_bar(stage), 0);
            tma_load_2d_pair(smem_a + stage * S::kABytes, &p.tmA[q], kb * kBK, m0, lead_full);
            tma_load_2d_pair(smem_b + stage * S::kBBytes, &p.tmB[q], kb * kBK, n0, lead_full);
          } else {
            mbar_arrive_expect_tx(full_bar(stage), S::kStageBytes);
            tma_load_2d(smem_a + stage * S::kABytes, &p.tmA[q], kb * kBK, m0, full_bar(stage));
            tma_load_2d(smem_b + stage * S::kBBytes, &p.tmB[q], kb * kBK, n0, full_bar(stage));
          }
          issued_mask |= 1u << stage;
          last_parity = (last_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok && rank == 0) {
        // leave no copy in flight behind: wait (bounded) for every load issued
        for (int s = 0; s < kStages; ++s) {
          if (!(issued_mask & (1u << s))) continue;
          const uint64_t t0 = global_timer_ns();
          while (!mbar_try_wait(full_bar(s), (last_parity >> s) & 1u)) {
            if (global_timer_ns() - t0 > 1000000ull) break;
          }
        }
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer (of a pair: the leader only)
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int lt = 0;
      bool ok = true;
      for (int unit = first_unit; unit < total_tiles && ok; unit += unit_step) {
        if (skipped(unit % plain_tiles)) continue;
        const int iters = unit_iters(unit);
        const int buf = lt & 1;
        const uint32_t acc_phase = (lt >> 1) & 1;
        if (!mbar_wait_bounded(acc_empty_bar(buf), acc_phase ^ 1u, abort_flag, 2u, p.wait_limit_ns)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * BN);
        for (int it = 0; it < iters; ++it) {
          if (!mbar_wait_bounded(full_bar(stage), phase, abort_flag, 3u, p.wait_limit_ns)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint64_t a_desc = umma_desc_kmajor_sw128(smem_a + stage * S::kABytes, 1024);
          const uint64_t b_desc = umma_desc_kmajor_sw128(smem_b + stage * S::kBBytes, 1024);
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk) {
            // 16 k-elements = 32 bytes further along the swizzled row: +2 in address>>4 units
            if constexpr (CTAS == 2)
              tc_mma_bf16_pair(d_tmem, a_desc + 2u * kk, b_desc + 2u * kk, idesc, (it > 0 || kk > 0) ? 1u : 0u);
            else
              tc_mma_bf16(d_tmem, a_desc + 2u * kk, b_desc + 2u * kk, idesc, (it > 0 || kk > 0) ? 1u : 0u);
          }
          // frees the stage (in both CTAs of a pair) once these MMAs have read it
          if constexpr (CTAS == 2) tc_commit_pair(empty_bar(stage), 3); else tc_commit(empty_bar(stage));
          if (++stage == kStages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) {  // accumulator complete
          if constexpr (CTAS == 2) tc_commit_pair(acc_full_bar(buf), 3); else tc_commit(acc_full_bar(buf));
        }
        ++lt;
      }
    }
  } else {
    // ---------------------------------------------------------------- epilogue
    const int lane_group = warp & 3;  // a warp may touch only tensor-memory lanes 32*(warp%4)..+31
    // warps 2..5 take the left half of the tile's columns, warps 6..9 the right half: per-row records
    // (moments, quantisation error) are therefore per half tile, index 2 * n_tile + half
    constexpr int kHalf = BN / 2;
    const int half = (warp - 2) >> 2;
    const int cbeg = half * kHalf, cend = cbeg + kHalf;
    // the leader counts drained accumulators: the partner's warps arrive on the leader's barrier
    auto release_acc = [&](int b) {
      if constexpr (CTAS == 2) mbar_arrive_cluster(cluster_map_shared(acc_empty_bar(b), 0));
      else mbar_arrive(acc_empty_bar(b));
    };
    int lt = 0;
    bool ok = true;
    for (int unit = first_unit; unit < total_tiles && ok; unit += unit_step) {
      const int tile = unit % plain_tiles;
      if (skipped(tile)) continue;
      int m_tile, n_tile;
      tile_mn(tile, m_tile, n_tile);
      const int row = m_tile * kTileM + static_cast<int>(rank) * kBM + lane_group * 32 + lane;
      const int n0 = n_tile * BN;
      const int buf = lt & 1;
      const uint32_t acc_phase = (lt >> 1) & 1;
      // the tensor-memory loads below are warp-collective: the whole warp goes on or the whole warp leaves
      const bool got = mbar_wait_bounded(acc_full_bar(buf), acc_phase, abort_flag, 4u, p.wait_limit_ns);
      if (!__all_sync(0xffffffffu, got)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      const uint32_t t_addr =
          tmem_base + (static_cast<uint32_t>(lane_group * 32) << 16) + static_cast<uint32_t>(buf * BN);
      const bool row_ok = row < p.M;
      const bool scaled = p.row_scale != nullptr;  // uniform over the grid
      const float rs = (scaled && row_ok) ? p.row_scale[row] : 1.0f;
      auto scale32 = [&](uint32_t (&a)[32]) {
        if (scaled) {
#pragma unroll
          for (int j = 0; j < 32; ++j) a[j] = __float_as_uint(__uint_as_float(a[j]) * rs);
        }
      };
      uint32_t v[32];

      if constexpr (EPI == kStoreF32) {
#pragma unroll 1
        for (int c0 = cbeg; c0 < cend; c0 += 32) {
          tmem_ld_32x32(t_addr + c0, v);
          tc_wait_ld();
          scale32(v);
          if (row_ok)
            store_row32(p.out + static_cast<long long>(unit / plain_tiles) * p.split_stride +
                            static_cast<long long>(row) * p.ldo + n0 + c0,
                        v, p.out_sector_aligned != 0);
        }
      } else if constexpr (EPI == kMoments) {
        // The thread's half row (kHalf columns) is read into registers in one go and the accumulator goes back to the
        // MMA warp at once: the arithmetic and the stores below no longer sit between two tiles' MMAs.
        constexpr int kChunks = kHalf / 32;
        uint32_t vv[kChunks][32];
#pragma unroll
        for (int c = 0; c < kChunks; ++c) tmem_ld_32x32(t_addr + cbeg + 32 * c, vv[c]);
        tc_wait_ld();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) release_acc(buf);
        // With float16 operands the accumulator holds the product of rows scaled into [1, 2): the row factor is not
        // applied to the entries but to the results (the mean by f, the k-th central sum by f^k) and to the stored
        // copies on their way out (the float16 one takes it into its own factor), one multiplication per entry less.
        // With bf16 operands the accumulator carries X's own scale, and the factor (RMSNorm's) has to come first, so
        // that the fourth powers stay in range whatever that scale is.
        const bool pre = scaled && p.f16_operands == 0;
        if (pre) {
#pragma unroll
          for (int c = 0; c < kChunks; ++c) scale32(vv[c]);
        }
        const float post = (scaled && !pre) ? rs : 1.0f;
        // pass 1: mean of the kHalf columns; pass 2: central power sums about it
        float s1 = 0.f;
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            a0 += __uint_as_float(vv[c][j]);
            a1 += __uint_as_float(vv[c][j + 1]);
            a2 += __uint_as_float(vv[c][j + 2]);
            a3 += __uint_as_float(vv[c][j + 3]);
          }
          s1 += (a0 + a1) + (a2 + a3);
        }
        float mean = s1 * (1.0f / kHalf);
        float s2 = 0.f, s3 = 0.f, s4 = 0.f;
#pragma unroll
        for (int c = 0; c < kChunks; ++c) {
          float b2 = 0.f, b3 = 0.f, b4 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float cc = __uint_as_float(vv[c][j]) - mean;
            const float c2 = cc * cc;
            b2 += c2;
            b3 = fmaf(c2, cc, b3);
            b4 = fmaf(c2, c2, b4);
          }
          s2 += b2;
          s3 += b3;
          s4 += b4;
        }
        if (post != 1.0f) {   // (factor by factor: no power of f is formed that the result does not need)
          mean *= post;
          s2 = (s2 * post) * post;
          s3 = ((s3 * post) * post) * post;
          s4 = (((s4 * post) * post) * post) * post;
        }
        if (row_ok) p.partial[static_cast<long long>(2 * n_tile + half) * p.M + row] = make_float4(mean, s2, s3, s4);
        // keep the float32 tile for the backward pass (the caller's choice; see kt_config.backward_mode)
        if (p.out != nullptr && row_ok) {
#pragma unroll
          for (int c = 0; c < kChunks; ++c) {
            if (post != 1.0f) {
#pragma unroll
              for (int j = 0; j < 32; ++j) vv[c][j] = __float_as_uint(__uint_as_float(vv[c][j]) * post);
            }
            store_row32(p.out + static_cast<long long>(row) * p.ldo + n0 + cbeg + 32 * c, vv[c],
                        p.out_sector_aligned != 0);
          }
        }
        if (p.out16 != nullptr && row_ok) {
          // float16 copy of the half row for the backward pass.  |y| <= |mean| + |c| and c^2 <= sum of c^2:
          // with e the biased exponent of that bound (< 2^(e - 126)), 2^(140 - e) brings every entry below 2^14.
          // e is kept in [14, 254] so that both the factor and its inverse 2^(e - 140) are normal float32 numbers.
          const float bound = fabsf(mean) + sqrtf(s2);
          unsigned int e = (__float_as_uint(bound) >> 23) & 0xffu;
          e = e < 14u ? 14u : (e > 254u ? 254u : e);
          const float mul = __uint_as_float((267u - e) << 23) * post;   // (entries not yet scaled: post is their factor)
          p.out16_exp[static_cast<long long>(2 * n_tile + half) * p.M + row] = static_cast<unsigned char>(e);
          __half* dst = p.out16 + static_cast<long long>(row) * p.ldo + n0 + cbeg;
#pragma unroll
          for (int c = 0; c < kChunks; ++c) {
            uint32_t h[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const __half2 hh = __floats2half2_rn(__uint_as_float(vv[c][2 * j]) * mul,
                                                   __uint_as_float(vv[c][2 * j + 1]) * mul);
              h[j] = *reinterpret_cast<const uint32_t*>(&hh);
            }
            // (column offsets are multiples of 32 entries and the row pitch of 128 entries: 32-byte aligned)
            st_global_v8(reinterpret_cast<float*>(dst + 32 * c), h);
            st_global_v8(reinterpret_cast<float*>(dst + 32 * c + 16), h + 8);
          }
        }
      } else if constexpr (EPI == kGrad) {
        float4 cf = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row_ok) cf = p.coef[row];
        __nv_bfloat16* gcol = p.gt + static_cast<long long>(n0) * p.ldg + row;
#pragma unroll 1
        for (int c0 = cbeg; c0 < cend; c0 += 32) {
          tmem_ld_32x32(t_addr + c0, v);
          tc_wait_ld();
          scale32(v);
          if (row_ok) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float c = __uint_as_float(v[j]) - cf.x;
              // a c^3 - ab c - am3
              const float g = fmaf(c, fmaf(cf.y * c, c, -cf.z), -cf.w);
              gcol[static_cast<long long>(c0 + j) * p.ldg] = __float2bfloat16_rn(g);
            }
          }
        }
      } else if constexpr (EPI == kAbsMax) {
        const bool asym = p.rowmin != nullptr;
        float mx = asym ? -INFINITY : 0.f, mn = INFINITY;
#pragma unroll 1
        for (int c0 = cbeg; c0 < cend; c0 += 32) {
          tmem_ld_32x32(t_addr + c0, v);
          tc_wait_ld();
          scale32(v);
          if (asym) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float y = __uint_as_float(v[j]);
              mx = fmaxf(mx, y);
              mn = fminf(mn, y);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) mx = fmaxf(mx, fabsf(__uint_as_float(v[j])));
          }
        }
        // integer max/min of order-preserving bit patterns are exact: arrival order does not matter
        // (non-negative floats order like their own bits, which the symmetric case uses directly)
        if (row_ok) {
          if (asym) {
            atomicMax(p.rowmax + row, ordered_key(mx));
            atomicMin(p.rowmin + row, ordered_key(mn));
          } else {
            atomicMax(p.rowmax + row, __float_as_uint(mx));
          }
        }
      } else if constexpr (EPI == kQuantErr) {
        // Q(y) = clamp(round((y - b) / s), q_lo, q_hi) * s + b, every operation in IEEE float32
        float range = 0.f, b = 0.f;
        if (row_ok) {
          if (p.rowmin != nullptr) {
            const float hi = __fmul_rn(p.q_clip, ordered_value(p.rowmax[row]));
            b = __fmul_rn(p.q_clip, ordered_value(p.rowmin[row]));
            range = __fsub_rn(hi, b);
          } else {
            range = __fmul_rn(p.q_clip, __uint_as_float(p.rowmax[row]));
          }
        }
        const float s = __fdiv_rn(range, p.q_den);
        float e2 = 0.f;
#pragma unroll 1
        for (int c0 = cbeg; c0 < cend; c0 += 32) {
          tmem_ld_32x32(t_addr + c0, v);
          tc_wait_ld();
          scale32(v);
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float y = __uint_as_float(v[j]);
            float qv = 0.f;
            if (s > 0.f) {
              qv = rintf(__fdiv_rn(__fsub_rn(y, b), s));
              qv = fminf(fmaxf(qv, p.q_lo), p.q_hi);
            }
            const float e = __fsub_rn(y, __fadd_rn(__fmul_rn(qv, s), b));
            e2 = fmaf(e, e, e2);
          }
        }
        if (row_ok) p.qerr[static_cast<long long>(2 * n_tile + half) * p.M + row] = e2;
      }

      // hand the accumulator back to the MMA warp (kMoments did so as soon as it had the tile in registers)
      if constexpr (EPI != kMoments) {
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) release_acc(buf);
      }
      ++lt;
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before_sync();
  __syncthreads();
  if constexpr (CTAS == 2) cluster_sync_all();  // neither CTA frees tensor memory or leaves while its partner still works
  if (warp == 1) {
    __syncwarp();
    tc_fence_after_sync();
    if constexpr (CTAS == 2) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0 && *abort_flag != 0 && p.err_word != nullptr) atomicMax(p.err_word, *abort_flag);
}

// Test hook: one thread waits, through the same bounded wait as every kernel of this library, on a barrier that
// nobody ever arrives on.  The wait gives up after limit_ns, the kernel returns normally, and *err_word receives
// the waiting role's code (99): exactly what a stalled pipeline would leave behind.
__global__ void k_wait_probe(unsigned long long limit_ns, unsigned int* err_word) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) (void)mbar_wait_bounded(smem_u32(&bar), 0u, &abort_flag, 99u, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag != 0 && err_word != nullptr) atomicMax(err_word, abort_flag);
}

}  // namespace kt
