// bf16 x bf16 -> f32 GEMM on the 5th-generation tensor cores (tcgen05.mma with
// the accumulator in tensor memory, operands staged by TMA), used for the gate's
// projection [Q' | K' | V'] = X [Wq_g | Wk_g | Wv_g] (Sec. 3.3, MHA').
//
// One CTA computes MT (1 or 2) sub-tiles of 128 rows x BN columns (BN = 128, 192 or 256) of the packed output - or, for the tiles of a last wave that
// would fill less than half of the SMs, one half of it (each such tile goes to two CTAs of
// BN / 2 columns, so that the wave ends in about half the time).  Warp 0 drives TMA,
// warp 1 owns TMEM and issues the MMAs, warps 2..9 drain the accumulator (two per quarter of its lanes): the
// float32 form straight to global memory, the hi / lo bf16 form through the
// (by then free) operand stages and TMA stores, which write whole 128-byte lines.
//   A = X   [M, K]  row-major  -> K-major operand, 128-byte swizzled rows
//   B = W   [K, GD] row-major  -> MN-major operand: panels of [64 k][64 n]
// Products of bf16 inputs are exact in the f32 accumulator, so the result
// differs from an exact evaluation only by f32 summation error.
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

constexpr int kTcBM = 128, kTcBK = 64, kTcThreads = 320;   // warps: TMA, MMA, 8 x epilogue

// MT: 128-row sub-tiles of A per CTA (1 or 2; two share every B stage, a third less traffic per FLOP).
template <int BN, int MT> struct GemmTcCfg {
  static constexpr int kStages = BN == 256 ? (MT == 2 ? 3 : 4) : BN == 192 ? 4 : 6;
  static constexpr int kAccCols = BN > 128 ? 256 : 128;      // TMEM columns between the sub-tiles' accumulators
  static constexpr int kABytes = MT * kTcBM * kTcBK * 2;     // 16 KB per sub-tile
  static constexpr int kPanelBytes = kTcBK * 64 * 2;         // [64 k][64 n] = 8 KB
  static constexpr int kBBytes = (BN / 64) * kPanelBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
};

template <int BN, int MT>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_bf16_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                    const __grid_constant__ CUtensorMap tmChi, const __grid_constant__ CUtensorMap tmClo,
                    float *__restrict__ C, bool split, int M, int K, int GD, int n_tiles_n, int halved_from) {
  using Cfg = GemmTcCfg<BN, MT>;
  constexpr uint32_t kTmemCols = MT * Cfg::kAccCols;
  static_assert(kTmemCols == 128 || kTmemCols == 256 || kTmemCols == 512, "TMEM columns: a power of two");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + Cfg::kStages * Cfg::kStageBytes);
  uint64_t *empty = full + Cfg::kStages;
  uint64_t *acc_full = empty + Cfg::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  int *gave_up = reinterpret_cast<int *>(tmem_slot + 1);   // set by an epilogue thread whose wait for the accumulator expired

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTAs below halved_from take whole tiles (row-major over the tile grid), the rest half tiles
  const int cta = blockIdx.x;
  const bool halved = cta >= halved_from;
  const int tile = halved ? halved_from + ((cta - halved_from) >> 1) : cta;
  const int bn = halved ? BN / 2 : BN;         // columns of this CTA (a multiple of 64)
  const int m0 = (tile / n_tiles_n) * (MT * kTcBM);
  const int n0 = (tile % n_tiles_n) * BN + (halved ? ((cta - halved_from) & 1) * (BN / 2) : 0);   // in the packed [3 * GD] output
  // a 64-column panel of B lies in one weight (64 divides GD); a tile may straddle two
  const int num_kb = (K + kTcBK - 1) / kTcBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB0);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % Cfg::kStages;
        const uint32_t ph = (kb / Cfg::kStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1)) break;
        uint8_t *a = smem + s * Cfg::kStageBytes, *b = a + Cfg::kABytes;
        mbar_arrive_expect_tx(&full[s], Cfg::kABytes + (bn / 64) * Cfg::kPanelBytes);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)              // rows past M are filled with zeros
          tma_load_2d(a + mt * (kTcBM * kTcBK * 2), &tmA, &full[s], kb * kTcBK, m0 + mt * kTcBM);
        for (int p = 0; p < bn / 64; ++p) {
          const int col = n0 + p * 64, which = col / GD;
          tma_load_2d(b + p * Cfg::kPanelBytes, which == 0 ? &tmB0 : (which == 1 ? &tmB1 : &tmB2), &full[s],
                      col % GD, kb * kTcBK);
        }
      }
    }
  } else if (warp == 1) {
    // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
    const uint32_t idesc = idesc_bf16_f32(kTcBM, bn, false, true);
    const uint64_t da0 = desc_kmajor_sw128(smem_u32(smem));
    const uint64_t db0 = desc_mnmajor_sw128(smem_u32(smem) + Cfg::kABytes, Cfg::kPanelBytes);
    const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
    const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % Cfg::kStages;
      const uint32_t ph = (kb / Cfg::kStages) & 1;
      ok = mbar_wait(&full[s], ph);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t a_lo = a_lo0 + ((s * Cfg::kStageBytes) >> 4), b_lo = b_lo0 + ((s * Cfg::kStageBytes) >> 4);
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kTcBK / 16; ++k) {
          // 16 elements of K: 32 bytes along a K-major row; 16 k-rows (2048 B) of an MN-major panel
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            mma_ss_lohi(tmem_acc + mt * Cfg::kAccCols, a_lo + ((mt * kTcBM * kTcBK * 2 + k * 32) >> 4), a_hi,
                        b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
        }
        mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
      }
      __syncwarp();
    }
    if (elect_one()) mma_commit(acc_full);   // accumulator complete (or unwinding)
    __syncwarp();
  } else {
    // epilogue: warp w may touch TMEM lanes [32 * (w % 4), +32); warps 2..5 drain the first half of
    // the tile's columns, warps 6..9 the second
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int c_begin = half * (bn / 2), c_end = c_begin + bn / 2;      // bn / 2 is a multiple of 32
    // all eight warps agree on whether the accumulator arrived before any of them enters the barriers below
    if (!mbar_wait(acc_full, 0)) *gave_up = 1;
    named_barrier_sync(1, 256);
    const bool ok = *gave_up == 0;
    tc_fence_after_sync();
#pragma unroll 1
    for (int mt = 0; mt < MT; ++mt) {
    const int row = m0 + mt * kTcBM + quad * 32 + lane;
    const uint32_t tmem_sub = tmem_acc + mt * Cfg::kAccCols;
    if (ok && num_kb > 0 && split) {
      // x = hi + lo in bf16 pairs, for consumers that rebuild float32 precision from three
      // products.  Every MMA has completed, so every stage has been read: the tile is staged
      // over them as panels of [128 rows][64 bf16] (128-byte rows, 16-byte chunks XOR-swizzled by
      // the row, the layout of a swizzled TMA store): hi panels first, then lo panels.
      static_assert(2 * (BN / 64) * kTcBM * 128 <= Cfg::kStages * Cfg::kStageBytes, "staging fits the stages");
      const int r_in = quad * 32 + lane;
      uint8_t *stage_lo = smem + (BN / 64) * kTcBM * 128;
#pragma unroll 1
      for (int c = c_begin; c < c_end; c += 32) {
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_sub + ((uint32_t)(quad * 32) << 16) + c, r);
        const uint32_t panel = (uint32_t)(c >> 6) * kTcBM * 128 + r_in * 128;
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint32_t h[4], l[4];
#pragma unroll
          for (int q = 0; q < 8; q += 2) {
            float h0, l0, h1, l1;
            split_bf16(__uint_as_float(r[e + q]), h0, l0);
            split_bf16(__uint_as_float(r[e + q + 1]), h1, l1);
            h[q >> 1] = pack_bf16x2(h0, h1);
            l[q >> 1] = pack_bf16x2(l0, l1);
          }
          const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + (e >> 3));          // 16-byte chunk within the 128-byte row
          const uint32_t off = panel + ((chunk ^ (r_in & 7)) << 4);
          *reinterpret_cast<uint4 *>(smem + off) = make_uint4(h[0], h[1], h[2], h[3]);
          *reinterpret_cast<uint4 *>(stage_lo + off) = make_uint4(l[0], l[1], l[2], l[3]);
        }
      }
      fence_proxy_async_smem();
      named_barrier_sync(1, 256);
      if (threadIdx.x == 64) {
        for (int p = 0; p < bn / 64; ++p) {            // rows past M are dropped by the tensor map
          tma_store_2d(&tmChi, smem + p * kTcBM * 128, n0 + p * 64, m0 + mt * kTcBM);
          tma_store_2d(&tmClo, stage_lo + p * kTcBM * 128, n0 + p * 64, m0 + mt * kTcBM);
        }
        tma_store_commit();
        tma_store_wait_read();
      }
      if (MT > 1) named_barrier_sync(1, 256);          // the staging area is free for the next sub-tile
    } else if (ok && num_kb > 0) {
      const size_t crow = (size_t)row * 3 * GD + n0;
#pragma unroll 1
      for (int c = c_begin; c < c_end; c += 32) {
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_sub + ((uint32_t)(quad * 32) << 16) + c, r);
        if (row < M) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4 *>(C + crow + c + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
        }
      }
    }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (cta_group::2): a pair computes 256 rows x 384 columns, each CTA holding
// its 128 rows of X and half of every stage of W; the leader issues, per 16 elements of K, one MMA of
// M = 256, N = 256 and one of N = 128 (384 = 3 x 128 divides the packed width 3 GD of every shape
// this file covers).  Per 64-deep k-block the tensor cores read 56 KB of operands from each CTA's
// shared memory while TMA writes 40 KB, under the 128 bytes a clock shared memory moves in the 768
// clocks of MMA work; one CTA on a 256 x 192 tile (the same work) moves 136 KB and takes ~1,050.
// The whole tile is staged at once over the operand stages (hi and lo: 192 KB of the 200).
constexpr int kGpBN = 384, kGpStages = 5;
constexpr int kGpABytes = kTcBM * kTcBK * 2;                      // 16 KB: this CTA's rows of X
constexpr int kGpPanelBytes = kTcBK * 64 * 2;                     // [64 k][64 n] = 8 KB
constexpr int kGpBBytes = (kGpBN / 2 / 64) * kGpPanelBytes;       // 24 KB: two panels of the N = 256 MMA, one of the N = 128
constexpr int kGpStageBytes = kGpABytes + kGpBBytes;              // 40 KB
constexpr int kGpSmemBytes = kGpStages * kGpStageBytes + 1024 + 256;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTcThreads, 1)
gemm_bf16_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                      const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                      const __grid_constant__ CUtensorMap tmChi, const __grid_constant__ CUtensorMap tmClo,
                      float *__restrict__ C, bool split, int M, int K, int GD, int n_tiles_n) {
  constexpr uint32_t kTmemCols = 512;              // 384 used: columns [0, 256) of the wide MMA, [256, 384) of the narrow
  static_assert(2 * (kGpBN / 64) * kTcBM * 128 <= kGpStages * kGpStageBytes, "staging fits the stages");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kGpStages * kGpStageBytes);   // used in the leader only
  uint64_t *empty = full + kGpStages;              // one set per CTA: a commit arrives on both
  uint64_t *acc_full = empty + kGpStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  int *gave_up = reinterpret_cast<int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();         // 0: leader
  const int tile = blockIdx.x >> 1;
  const int m0 = (tile / n_tiles_n) * (2 * kTcBM) + (int)rank * kTcBM;   // this CTA's rows
  const int n0 = (tile % n_tiles_n) * kGpBN;                              // in the packed [3 * GD] output
  const int num_kb = (K + kTcBK - 1) / kTcBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGpStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB0);
  }
  __syncthreads();
  if (warp == 1) {                                 // the same warp of both CTAs, the same arguments
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  cluster_arrive_wait();                           // both CTAs' barriers are initialised, tensor memory is allocated
  tc_fence_after_sync();
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kGpStages;
        const uint32_t ph = (kb / kGpStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1)) break;  // this CTA's copy: the MMAs that read the stage (in both CTAs) are done
        uint8_t *a = smem + s * kGpStageBytes, *b = a + kGpABytes;
        if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * kGpStageBytes);   // the leader's barrier counts both CTAs' bytes
        const uint32_t bar = mapa_shared(smem_u32(&full[s]), 0);
        tma_load_2d_pair(a, &tmA, bar, kb * kTcBK, m0);                      // rows past M are filled with zeros
#pragma unroll
        for (int p = 0; p < 3; ++p) {
          // this CTA's half of the wide MMA's columns (two panels), then of the narrow one's (one panel);
          // a 64-column panel lies in one weight (64 divides GD)
          const int col = n0 + (p < 2 ? (int)rank * 128 + p * 64 : 256 + (int)rank * 64), which = col / GD;
          tma_load_2d_pair(b + p * kGpPanelBytes, which == 0 ? &tmB0 : (which == 1 ? &tmB1 : &tmB2), bar, col % GD,
                           kb * kTcBK);
        }
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {
      // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
      const uint32_t idesc_w = idesc_bf16_f32(2 * kTcBM, 256, false, true), idesc_n = idesc_bf16_f32(2 * kTcBM, 128, false, true);
      const uint64_t da0 = desc_kmajor_sw128(smem_u32(smem));
      const uint64_t db0 = desc_mnmajor_sw128(smem_u32(smem) + kGpABytes, kGpPanelBytes);
      const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
      const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % kGpStages;
        const uint32_t ph = (kb / kGpStages) & 1;
        ok = mbar_wait(&full[s], ph);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a_lo = a_lo0 + ((s * kGpStageBytes) >> 4), b_lo = b_lo0 + ((s * kGpStageBytes) >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k) {
            // 16 elements of K: 32 bytes along a K-major row; 16 k-rows (2048 B) of an MN-major panel
            mma_ss_pair_lohi(tmem_acc, a_lo + ((k * 32) >> 4), a_hi, b_lo + ((k * 2048) >> 4), b_hi, idesc_w, (kb | k) != 0);
            mma_ss_pair_lohi(tmem_acc + 256, a_lo + ((k * 32) >> 4), a_hi, b_lo + ((2 * kGpPanelBytes + k * 2048) >> 4), b_hi,
                             idesc_n, (kb | k) != 0);
          }
          mma_commit_pair(&empty[s]);              // frees the stage in both CTAs once these MMAs have read it
        }
        __syncwarp();
      }
      if (elect_one()) mma_commit_pair(acc_full);  // accumulators complete (or unwinding), in both CTAs
      __syncwarp();
    }
  } else {
    // epilogue: warp w may touch TMEM lanes [32 * (w % 4), +32); warps 2..5 drain columns [0, 192), warps 6..9 the rest
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int c_begin = half * (kGpBN / 2), c_end = c_begin + kGpBN / 2;
    if (!mbar_wait(acc_full, 0)) *gave_up = 1;
    named_barrier_sync(1, 256);
    const bool ok = *gave_up == 0;
    tc_fence_after_sync();
    const int r_in = quad * 32 + lane, row = m0 + r_in;
    if (ok && num_kb > 0 && split) {
      // x = hi + lo in bf16 pairs.  Every MMA of both CTAs has completed, so every stage has been read: the
      // tile is staged over them as panels of [128 rows][64 bf16] (128-byte rows, 16-byte chunks
      // XOR-swizzled by the row): six hi panels, then six lo panels.
      uint8_t *stage_lo = smem + (kGpBN / 64) * kTcBM * 128;
#pragma unroll 1
      for (int c = c_begin; c < c_end; c += 32) {
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_acc + ((uint32_t)(quad * 32) << 16) + c, r);
        const uint32_t panel = (uint32_t)(c >> 6) * kTcBM * 128 + r_in * 128;
#pragma unroll
        for (int e = 0; e < 32; e += 8) {
          uint32_t h[4], l[4];
#pragma unroll
          for (int q = 0; q < 8; q += 2) {
            float h0, l0, h1, l1;
            split_bf16(__uint_as_float(r[e + q]), h0, l0);
            split_bf16(__uint_as_float(r[e + q + 1]), h1, l1);
            h[q >> 1] = pack_bf16x2(h0, h1);
            l[q >> 1] = pack_bf16x2(l0, l1);
          }
          const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + (e >> 3));          // 16-byte chunk within the 128-byte row
          const uint32_t off = panel + ((chunk ^ (r_in & 7)) << 4);
          *reinterpret_cast<uint4 *>(smem + off) = make_uint4(h[0], h[1], h[2], h[3]);
          *reinterpret_cast<uint4 *>(stage_lo + off) = make_uint4(l[0], l[1], l[2], l[3]);
        }
      }
      fence_proxy_async_smem();
      named_barrier_sync(1, 256);
      if (threadIdx.x == 64) {
        for (int p = 0; p < kGpBN / 64; ++p) {         // rows past M are dropped by the tensor map
          tma_store_2d(&tmChi, smem + p * kTcBM * 128, n0 + p * 64, m0);
          tma_store_2d(&tmClo, stage_lo + p * kTcBM * 128, n0 + p * 64, m0);
        }
        tma_store_commit();
        tma_store_wait_read();
      }
    } else if (ok && num_kb > 0) {
      const size_t crow = (size_t)row * 3 * GD + n0;
#pragma unroll 1
      for (int c = c_begin; c < c_end; c += 32) {
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_acc + ((uint32_t)(quad * 32) << 16) + c, r);
        if (row < M) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4 *>(C + crow + c + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
        }
      }
    }
  }
  // neither CTA leaves (or frees tensor memory) while the other may still use its shared or tensor memory
  tc_fence_before_sync();
  cluster_arrive_wait();
  if (warp == 1) tmem_dealloc_pair(tmem_acc, kTmemCols);
}

// ------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

int make_tmap_2d_bf16(CUtensorMap *out, const void *base, uint64_t rows, uint64_t cols, uint64_t pitch_bytes,
                      uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) { set_last_cuda_error((int)cudaErrorNotSupported); return AG_ERR_CUDA; }
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_last_cuda_error(1000 + (int)r); return AG_ERR_CUDA; }
  return AG_OK;
}

int make_tmap_3d_bf16(CUtensorMap *out, const void *base, uint64_t planes, uint64_t rows, uint64_t cols,
                      uint32_t box_rows, uint32_t box_cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) { set_last_cuda_error((int)cudaErrorNotSupported); return AG_ERR_CUDA; }
  cuuint64_t dims[3] = {cols, rows, planes};
  cuuint64_t strides[2] = {cols * 2, rows * cols * 2};
  cuuint32_t box[3] = {box_cols, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { set_last_cuda_error(1000 + (int)r); return AG_ERR_CUDA; }
  return AG_OK;
}

// ----------------------------------------------------------------- launch
static int gemm_sm_count() {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, v = 0;
    sms = (cudaGetDevice(&dev) == cudaSuccess &&
           cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) ? v : 148;
  }
  return sms;
}

template <int BN, int MT>
static int run_gemm_tc(const void *X, const void *W0, const void *W1, const void *W2, float *C,
                       __nv_bfloat16 *Chi, __nv_bfloat16 *Clo, int M, int K, int GD, cudaStream_t st) {
  using Cfg = GemmTcCfg<BN, MT>;
  CUtensorMap tmA, tmB[3];
  int rc = make_tmap_2d_bf16(&tmA, X, M, K, (uint64_t)K * 2, kTcBM, kTcBK);
  if (rc) return rc;
  const void *Ws[3] = {W0, W1, W2};
  for (int i = 0; i < 3; ++i) {
    rc = make_tmap_2d_bf16(&tmB[i], Ws[i], K, GD, (uint64_t)GD * 2, kTcBK, 64);
    if (rc) return rc;
  }
  // output maps of the hi / lo form (one row of a weight stands in when that form is not asked for)
  CUtensorMap tmC[2];
  const void *outs[2] = {Chi ? (const void *)Chi : W0, Clo ? (const void *)Clo : W0};
  for (int i = 0; i < 2; ++i) {
    rc = Chi ? make_tmap_2d_bf16(&tmC[i], outs[i], M, 3 * (uint64_t)GD, 3 * (uint64_t)GD * 2, kTcBM, 64)
             : make_tmap_2d_bf16(&tmC[i], outs[i], 1, GD, (uint64_t)GD * 2, 1, 64);
    if (rc) return rc;
  }
  auto kern = gemm_bf16_tc_kernel<BN, MT>;
  AG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
  const int n_tiles_n = 3 * GD / BN, n_tiles = n_tiles_n * ((M + MT * kTcBM - 1) / (MT * kTcBM));
  // tiles of a last wave that would fill at most half of the SMs are halved
  const int sms = gemm_sm_count();
  const int tail = n_tiles % sms;
  const int halved_from = (BN % 128 == 0 && tail > 0 && 2 * tail <= sms) ? n_tiles - tail : n_tiles;   // (any MT)
  const int ctas = halved_from + 2 * (n_tiles - halved_from);
  kern<<<ctas, kTcThreads, Cfg::kSmemBytes, st>>>(tmA, tmB[0], tmB[1], tmB[2], tmC[0], tmC[1], C, Chi != nullptr, M, K,
                                                  GD, n_tiles_n, halved_from);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

static int run_gemm_pair(const void *X, const void *W0, const void *W1, const void *W2, float *C, __nv_bfloat16 *Chi,
                         __nv_bfloat16 *Clo, int M, int K, int GD, cudaStream_t st) {
  CUtensorMap tmA, tmB[3];
  int rc = make_tmap_2d_bf16(&tmA, X, M, K, (uint64_t)K * 2, kTcBM, kTcBK);
  if (rc) return rc;
  const void *Ws[3] = {W0, W1, W2};
  for (int i = 0; i < 3; ++i) {
    rc = make_tmap_2d_bf16(&tmB[i], Ws[i], K, GD, (uint64_t)GD * 2, kTcBK, 64);
    if (rc) return rc;
  }
  CUtensorMap tmC[2];
  const void *outs[2] = {Chi ? (const void *)Chi : W0, Clo ? (const void *)Clo : W0};
  for (int i = 0; i < 2; ++i) {
    rc = Chi ? make_tmap_2d_bf16(&tmC[i], outs[i], M, 3 * (uint64_t)GD, 3 * (uint64_t)GD * 2, kTcBM, 64)
             : make_tmap_2d_bf16(&tmC[i], outs[i], 1, GD, (uint64_t)GD * 2, 1, 64);
    if (rc) return rc;
  }
  AG_CUDA_TRY(cudaFuncSetAttribute(gemm_bf16_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGpSmemBytes));
  const int n_tiles_n = 3 * GD / kGpBN, n_tiles_m = (M + 2 * kTcBM - 1) / (2 * kTcBM);
  gemm_bf16_pair_kernel<<<2 * n_tiles_n * n_tiles_m, kTcThreads, kGpSmemBytes, st>>>(
      tmA, tmB[0], tmB[1], tmB[2], tmC[0], tmC[1], C, Chi != nullptr, M, K, GD, n_tiles_n);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

bool gate_proj_tc_supported(int K, int GD) { return GD % 128 == 0 && K % 8 == 0; }

int launch_gate_proj_tc(const void *X, const void *W0, const void *W1, const void *W2, float *C, void *Chi,
                        void *Clo, int M, int K, int GD, cudaStream_t st) {
  auto hi = static_cast<__nv_bfloat16 *>(Chi), lo = static_cast<__nv_bfloat16 *>(Clo);
  // at least half a wave of pair tiles (256 x 384): CTA pairs
  if ((long long)(3 * GD / kGpBN) * ((M + 2 * kTcBM - 1) / (2 * kTcBM)) * 4 >= gemm_sm_count())
    return run_gemm_pair(X, W0, W1, W2, C, hi, lo, M, K, GD, st);
  if (GD % 256 == 0) {
    // more than one wave of 128 x 256 tiles: 256 x 256 tiles, whose two row sub-tiles share every
    // stage of W (a third less operand traffic per FLOP; the kernel is bound by feeding the SMs)
    const long long tiles128 = (long long)(3 * GD / 256) * ((M + kTcBM - 1) / kTcBM);
    if (tiles128 > gemm_sm_count()) {
      // one round either way: 192-column tiles put more SMs to work (the 7B-shaped layer: 128 tiles
      // of 256 x 192 instead of 96 of 256 x 256).  The time of a tile hardly depends on its width (the
      // operand loads, not the MMAs, set it), so with several rounds the fewer, wider tiles stay.
      const long long row_tiles = (M + 2 * kTcBM - 1) / (2 * kTcBM);
      if (GD % 64 == 0 && row_tiles * (3 * GD / 192) <= gemm_sm_count())
        return run_gemm_tc<192, 2>(X, W0, W1, W2, C, hi, lo, M, K, GD, st);
      return run_gemm_tc<256, 2>(X, W0, W1, W2, C, hi, lo, M, K, GD, st);
    }
    return run_gemm_tc<256, 1>(X, W0, W1, W2, C, hi, lo, M, K, GD, st);
  }
  return run_gemm_tc<128, 1>(X, W0, W1, W2, C, hi, lo, M, K, GD, st);
}

int gemm_tc_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
