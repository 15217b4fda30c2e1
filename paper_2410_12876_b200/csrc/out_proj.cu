// Output projection of the layer, Eq. 1: MHA(X) = [H_1(X), ..., H_h(X)] W^O, with the skip
// connection a stack of attention layers adds (Y = X + MHA(X)), on the 5th-generation tensor cores.
//
// The heads' outputs arrive as the prefill attention wrote them, O [B, h, n, D]: the concatenation
// of Eq. 1 is never materialised.  Token (b, t) of the GEMM's A operand is row t of the planes
// b h .. b h + h - 1 of O, so a 64-wide K block lies in one head and is fetched by a 3-D TMA box
// [1 plane][128 tokens][64 columns].  B = W^O [h D, d] is MN-major (panels of [64 k][64 n]).
//
// One CTA computes MT sub-tiles of 128 tokens x BN output columns.  Warp 0 drives TMA, warp 1 owns
// tensor memory and issues the MMAs, warps 2..9 drain the accumulator (two per quarter of its
// lanes): they fetch their rows of the skip connection into registers while the MMAs run (slice by
// slice, each released by the MMA warp, so that the fetch is neither one burst among the first
// operand loads nor waited for at the end), add them to the float32 accumulator, round once to
// bf16, stage the tile over the freed operand stages and send it off with TMA stores.  Tile order
// in bands of row tiles (the CTAs in flight share a few column slices of W^O while the band's rows
// of O stay in L2).
//
// out_proj_pair_kernel is the same GEMM on CTA pairs (cta_group::2), used when the tiles fill the
// SMs more than once.  out_proj_simt_kernel is the CUDA-core form for float32 layers, head_dim 64
// and shapes the tiles do not cover.
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

namespace {

constexpr int kBM = 128, kBK = 64, kThreads = 320, kD = 128;   // warps: TMA, MMA, 8 x epilogue
constexpr int kBandTiles = 16;
// The skip connection is fetched by the epilogue warps in slices of 32 columns spread over the main loop: slice i
// once the MMAs of k-block kMidKb + i * step are done.  Fetched as one burst (at the start, or when the
// accumulator is complete) it competes with the operand loads or is waited for.
constexpr int kMidKb = 4, kMaxSlices = 8;

template <int BN, int MT> struct OpCfg {
  static constexpr int kStages = BN == 256 ? (MT == 2 ? 3 : 4) : 6;
  static constexpr int kABytes = MT * kBM * kBK * 2;
  static constexpr int kPanelBytes = kBK * 64 * 2;           // [64 k][64 n] = 8 KB
  static constexpr int kBBytes = (BN / 64) * kPanelBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/;
};

template <int BN, int MT>
__global__ void __launch_bounds__(kThreads, 1)
out_proj_tc_kernel(const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmW,
                   const __grid_constant__ CUtensorMap tmY, const __nv_bfloat16 *__restrict__ X_res, int n_sub, int tps,
                   int n, int heads, int d, int n_tiles_m, int n_tiles_n) {
  using Cfg = OpCfg<BN, MT>;
  constexpr uint32_t kTmemCols = MT * BN;
  static_assert(kTmemCols == 128 || kTmemCols == 256 || kTmemCols == 512, "TMEM columns: a power of two");
  static_assert(MT * (BN / 64) * kBM * 128 <= Cfg::kStages * Cfg::kStageBytes, "staging fits the stages");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + Cfg::kStages * Cfg::kStageBytes);
  uint64_t *empty = full + Cfg::kStages;
  uint64_t *acc_full = empty + Cfg::kStages;
  uint64_t *sig = acc_full + 1;                   // kMaxSlices barriers that release the skip connection slice by slice
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sig + kMaxSlices);
  int *gave_up = reinterpret_cast<int *>(tmem_slot + 1);   // set by an epilogue thread whose wait for the accumulator expired

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x;
  const int band = tile / (kBandTiles * n_tiles_n), in_band = tile % (kBandTiles * n_tiles_n);
  const int band_rows = min(kBandTiles, n_tiles_m - band * kBandTiles);
  const int tile_m = band * kBandTiles + in_band % band_rows, tile_n = in_band / band_rows;
  // Rows are counted in sub-tiles of 128 tokens laid out per sequence: sequence b owns sub-tiles
  // [b tps, (b + 1) tps), the last of which may reach past the sequence's end (zeros on the way in,
  // dropped on the way out), so a sub-tile never spans two sequences.
  const int sub0 = tile_m * MT;
  const int n0 = tile_n * BN;
  const int num_kb = heads * (kD / kBK);         // K = h D, 64 at a time: two blocks per head
  const int sig_step = max(0, (num_kb - kMidKb - 8) / kMaxSlices);   // slice i leaves after k-block kMidKb + i sig_step

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    for (int i = 0; i < kMaxSlices; ++i) mbar_init(&sig[i], 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmO);
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmY);
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
        mbar_arrive_expect_tx(&full[s], Cfg::kStageBytes);
        const int head = kb / (kD / kBK), col = (kb % (kD / kBK)) * kBK;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          // tokens past the sequence's end, and whole sub-tiles past the batch, are filled with zeros
          const int sub = sub0 + mt, b_seq = sub / tps, t0 = (sub % tps) * kBM;
          tma_load_3d(a + mt * (kBM * kBK * 2), &tmO, &full[s], col, t0, b_seq * heads + head);
        }
#pragma unroll
        for (int p = 0; p < BN / 64; ++p)
          tma_load_2d(b + p * Cfg::kPanelBytes, &tmW, &full[s], n0 + p * 64, kb * kBK);
      }
    }
  } else if (warp == 1) {
    // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
    const uint32_t idesc = idesc_bf16_f32(kBM, BN, false, true);
    const uint64_t da0 = desc_kmajor_sw128(smem_u32(smem));
    const uint64_t db0 = desc_mnmajor_sw128(smem_u32(smem) + Cfg::kABytes, Cfg::kPanelBytes);
    const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
    const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
    bool ok = true;
    int nsig = 0;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % Cfg::kStages;
      const uint32_t ph = (kb / Cfg::kStages) & 1;
      ok = mbar_wait(&full[s], ph);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t a_lo = a_lo0 + ((s * Cfg::kStageBytes) >> 4), b_lo = b_lo0 + ((s * Cfg::kStageBytes) >> 4);
      int upto = nsig;                     // slices of the skip connection released after this k-block
      while (upto < kMaxSlices && kb >= min(num_kb - 1, kMidKb + upto * sig_step)) ++upto;
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            mma_ss_lohi(tmem_acc + mt * BN, a_lo + ((mt * kBM * kBK * 2 + k * 32) >> 4), a_hi,
                        b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
        }
        mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
        for (int i = nsig; i < upto; ++i) mma_commit(&sig[i]);
      }
      nsig = upto;
      __syncwarp();
    }
    if (elect_one()) {
      for (int i = nsig; i < kMaxSlices; ++i) mma_commit(&sig[i]);
      mma_commit(acc_full);                  // accumulator complete (or unwinding)
    }
    __syncwarp();
  } else {
    // epilogue warps: warp w may touch TMEM lanes [32 * (w % 4), +32); warps 2..5 drain the first
    // half of a sub-tile's columns, warps 6..9 the second
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int r_in = quad * 32 + lane;           // token of the sub-tile this thread drains
    constexpr int kChunks = BN / 2 / 32;         // 32-column chunks per thread and sub-tile
    // this thread's pieces of the skip connection, fetched while the MMAs run
    uint4 res[MT][kChunks][4];
    auto fetch_residual = [&](int mt, int ci) {
      const int sub = sub0 + mt, t = (sub % tps) * kBM + r_in;
      const bool have = X_res != nullptr && sub < n_sub && t < n;
      const size_t row = (size_t)(sub / tps) * n + t;
      const int c = half * (BN / 2) + ci * 32;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        res[mt][ci][q] = have ? ldg128_stream(X_res + row * d + n0 + c + q * 8) : make_uint4(0, 0, 0, 0);
    };
    bool fetched = true;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        fetched = fetched && mbar_wait(&sig[mt * kChunks + ci], 0);
        if (fetched) fetch_residual(mt, ci);
      }
    }
    if (!fetched) *gave_up = 1;
    // all eight warps agree on whether the accumulator arrived before any of them enters the barriers below
    if (!mbar_wait(acc_full, 0)) *gave_up = 1;
    named_barrier_sync(1, 256);
    const bool ok = *gave_up == 0;
    tc_fence_after_sync();
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int sub = sub0 + mt;
      if (!ok || sub >= n_sub) break;              // the same for all 256 threads
      const uint32_t tmem_sub = tmem_acc + mt * BN;
      // bf16 tile as panels of [128 tokens][64 columns] (128-byte rows, 16-byte chunks XOR-swizzled by the
      // row); each sub-tile has a staging area of its own, so the second is drained while the first leaves
      uint8_t *stg = smem + mt * (BN / 64) * kBM * 128;
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        const int c = half * (BN / 2) + ci * 32;
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_sub + ((uint32_t)(quad * 32) << 16) + c, r);
        const uint32_t panel = (uint32_t)(c >> 6) * kBM * 128 + r_in * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float xf[8];
          Elem<__nv_bfloat16>::unpack(res[mt][ci][q], xf);
          uint32_t h[4];
#pragma unroll
          for (int e = 0; e < 8; e += 2)
            h[e >> 1] = pack_bf16x2(__uint_as_float(r[q * 8 + e]) + xf[e], __uint_as_float(r[q * 8 + e + 1]) + xf[e + 1]);
          const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + q);
          *reinterpret_cast<uint4 *>(stg + panel + ((chunk ^ (r_in & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        }
      }
      fence_proxy_async_smem();
      named_barrier_sync(1, 256);                  // the tile is staged
      if (threadIdx.x == 64) {
#pragma unroll
        for (int p = 0; p < BN / 64; ++p)          // rows past the sequence's end are dropped by the tensor map
          tma_store_3d(&tmY, stg + p * kBM * 128, n0 + p * 64, (sub % tps) * kBM, sub / tps);
        tma_store_commit();
      }
    }
    if (threadIdx.x == 64) tma_store_wait_read();
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (cta_group::2): two CTAs on neighbouring SMs compute a 512-token x
// 256-column tile with shared MMAs of M = 256.  Each CTA holds two 128-token sub-tiles of A (its
// own 256 tokens) and ONE HALF of every W^O stage (128 of the 256 columns); an MMA reads A from
// both CTAs and half of B from each.  Per 64-deep k-block a CTA takes in 32 KB of A + 16 KB of B
// for 8.4 MFLOP, against 32 + 32 KB for the single-CTA tile: the operand loads, which pace that
// kernel, shrink by a quarter.  Loads are plain TMA loads (no multicast) that report to the
// leader's barrier; the leader (even CTA) issues the MMAs; a commit frees a stage in both CTAs.
constexpr int kPairBN = 256, kPairMT = 2, kPairStages = 4;
constexpr int kPairABytes = kPairMT * kBM * kBK * 2;                 // 32 KB: this CTA's two sub-tiles
constexpr int kPairBBytes = (kPairBN / 2 / 64) * (kBK * 64 * 2);     // 16 KB: this CTA's half of the W^O stage
constexpr int kPairBandTiles = 8;   // pair tiles of rows per band: the same 4096 tokens of A as a band of single-CTA tiles
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;           // 48 KB
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + 1024 + 256;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
out_proj_pair_kernel(const __grid_constant__ CUtensorMap tmO, const __grid_constant__ CUtensorMap tmW,
                     const __grid_constant__ CUtensorMap tmY, const __nv_bfloat16 *__restrict__ X_res, int n_sub, int tps,
                     int n, int heads, int d, int n_tiles_m, int n_tiles_n) {
  constexpr int BN = kPairBN, MT = kPairMT;
  constexpr uint32_t kTmemCols = MT * BN;          // 512: two accumulators of 128 rows x 256 columns per CTA
  static_assert(MT * (BN / 64) * kBM * 128 <= kPairStages * kPairStageBytes, "staging fits the stages");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kPairStages * kPairStageBytes);   // used in the leader only
  uint64_t *empty = full + kPairStages;            // one set per CTA: a commit arrives on both
  uint64_t *acc_full = empty + kPairStages;
  uint64_t *sig = acc_full + 1;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sig + kMaxSlices);
  int *gave_up = reinterpret_cast<int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();         // 0: leader
  const int tile = blockIdx.x >> 1;
  const int band = tile / (kPairBandTiles * n_tiles_n), in_band = tile % (kPairBandTiles * n_tiles_n);
  const int band_rows = min(kPairBandTiles, n_tiles_m - band * kPairBandTiles);
  const int tile_m = band * kPairBandTiles + in_band % band_rows, tile_n = in_band / band_rows;
  const int sub0 = tile_m * (2 * MT) + (int)rank * MT;   // this CTA's first sub-tile of 128 tokens
  const int n0 = tile_n * BN;
  const int num_kb = heads * (kD / kBK);
  const int sig_step = max(0, (num_kb - kMidKb - 8) / kMaxSlices);   // slice i leaves after k-block kMidKb + i sig_step

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    for (int i = 0; i < kMaxSlices; ++i) mbar_init(&sig[i], 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmO);
    prefetch_tensormap(&tmW);
    prefetch_tensormap(&tmY);
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
        const int s = kb % kPairStages;
        const uint32_t ph = (kb / kPairStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1)) break;  // this CTA's copy: the MMAs that read the stage (in both CTAs) are done
        uint8_t *a = smem + s * kPairStageBytes, *b = a + kPairABytes;
        // the leader's barrier counts the bytes of both CTAs
        if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * kPairStageBytes);
        const uint32_t bar = mapa_shared(smem_u32(&full[s]), 0);
        const int head = kb / (kD / kBK), col = (kb % (kD / kBK)) * kBK;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          // tokens past the sequence's end, and whole sub-tiles past the batch, are filled with zeros
          const int sub = sub0 + mt, b_seq = sub / tps, t0 = (sub % tps) * kBM;
          tma_load_3d_pair(a + mt * (kBM * kBK * 2), &tmO, bar, col, t0, b_seq * heads + head);
        }
#pragma unroll
        for (int p = 0; p < BN / 2 / 64; ++p)      // this CTA's half of the tile's columns
          tma_load_2d_pair(b + p * (kBK * 64 * 2), &tmW, bar, n0 + (int)rank * (BN / 2) + p * 64, kb * kBK);
      }
    }
  } else if (warp == 1) {
    if (rank == 0) {
      // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
      const uint32_t idesc = idesc_bf16_f32(2 * kBM, BN, false, true);
      const uint64_t da0 = desc_kmajor_sw128(smem_u32(smem));
      const uint64_t db0 = desc_mnmajor_sw128(smem_u32(smem) + kPairABytes, kBK * 64 * 2);
      const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
      const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
      bool ok = true;
      int nsig = 0;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % kPairStages;
        const uint32_t ph = (kb / kPairStages) & 1;
        ok = mbar_wait(&full[s], ph);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a_lo = a_lo0 + ((s * kPairStageBytes) >> 4), b_lo = b_lo0 + ((s * kPairStageBytes) >> 4);
        int upto = nsig;
        while (upto < kMaxSlices && kb >= min(num_kb - 1, kMidKb + upto * sig_step)) ++upto;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              mma_ss_pair_lohi(tmem_acc + mt * BN, a_lo + ((mt * kBM * kBK * 2 + k * 32) >> 4), a_hi,
                               b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
          }
          mma_commit_pair(&empty[s]);              // frees the stage in both CTAs once these MMAs have read it
          for (int i = nsig; i < upto; ++i) mma_commit_pair(&sig[i]);
        }
        nsig = upto;
        __syncwarp();
      }
      if (elect_one()) {
        for (int i = nsig; i < kMaxSlices; ++i) mma_commit_pair(&sig[i]);
        mma_commit_pair(acc_full);               // accumulators complete (or unwinding), in both CTAs
      }
      __syncwarp();
    }
  } else {
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int r_in = quad * 32 + lane;
    constexpr int kChunks = BN / 2 / 32;
    uint4 res[MT][kChunks][4];
    auto fetch_residual = [&](int mt, int ci) {
      const int sub = sub0 + mt, t = (sub % tps) * kBM + r_in;
      const bool have = X_res != nullptr && sub < n_sub && t < n;
      const size_t row = (size_t)(sub / tps) * n + t;
      const int c = half * (BN / 2) + ci * 32;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        res[mt][ci][q] = have ? ldg128_stream(X_res + row * d + n0 + c + q * 8) : make_uint4(0, 0, 0, 0);
    };
    bool fetched = true;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        fetched = fetched && mbar_wait(&sig[mt * kChunks + ci], 0);
        if (fetched) fetch_residual(mt, ci);
      }
    }
    if (!fetched) *gave_up = 1;
    if (!mbar_wait(acc_full, 0)) *gave_up = 1;
    named_barrier_sync(1, 256);
    const bool ok = *gave_up == 0;
    tc_fence_after_sync();
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int sub = sub0 + mt;
      if (!ok || sub >= n_sub) break;              // the same for all 256 threads
      const uint32_t tmem_sub = tmem_acc + mt * BN;
      uint8_t *stg = smem + mt * (BN / 64) * kBM * 128;
#pragma unroll
      for (int ci = 0; ci < kChunks; ++ci) {
        const int c = half * (BN / 2) + ci * 32;
        uint32_t r[32];
        tmem_ld_x32_sync(tmem_sub + ((uint32_t)(quad * 32) << 16) + c, r);
        const uint32_t panel = (uint32_t)(c >> 6) * kBM * 128 + r_in * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          float xf[8];
          Elem<__nv_bfloat16>::unpack(res[mt][ci][q], xf);
          uint32_t h[4];
#pragma unroll
          for (int e = 0; e < 8; e += 2)
            h[e >> 1] = pack_bf16x2(__uint_as_float(r[q * 8 + e]) + xf[e], __uint_as_float(r[q * 8 + e + 1]) + xf[e + 1]);
          const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + q);
          *reinterpret_cast<uint4 *>(stg + panel + ((chunk ^ (r_in & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        }
      }
      fence_proxy_async_smem();
      named_barrier_sync(1, 256);
      if (threadIdx.x == 64) {
#pragma unroll
        for (int p = 0; p < BN / 64; ++p)
          tma_store_3d(&tmY, stg + p * kBM * 128, n0 + p * 64, (sub % tps) * kBM, sub / tps);
        tma_store_commit();
      }
    }
    if (threadIdx.x == 64) tma_store_wait_read();
  }
  // neither CTA leaves (or frees tensor memory) while the other may still use its shared or tensor memory
  tc_fence_before_sync();
  cluster_arrive_wait();
  if (warp == 1) tmem_dealloc_pair(tmem_acc, kTmemCols);
}

int sm_count() {
  static int sms = 0;
  if (sms == 0) {
    int dev = 0, v = 0;
    sms = (cudaGetDevice(&dev) == cudaSuccess &&
           cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) ? v : 148;
  }
  return sms;
}

template <int BN, int MT>
int run_tc(const ag_layer_desc &dsc, const void *O, const void *Wo, const void *X_res, void *Y, cudaStream_t st) {
  using Cfg = OpCfg<BN, MT>;
  const int d = dsc.hidden, Kdim = dsc.heads * kD;
  const int tps = (dsc.seq + kBM - 1) / kBM, n_sub = dsc.batch * tps;   // sub-tiles of 128 tokens per sequence, in all
  CUtensorMap tmO, tmW, tmY;
  int rc = make_tmap_3d_bf16(&tmO, O, (uint64_t)dsc.batch * dsc.heads, dsc.seq, kD, kBM, kBK);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmW, Wo, Kdim, d, (uint64_t)d * 2, kBK, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmY, Y, dsc.batch, dsc.seq, d, kBM, 64);
  if (rc) return rc;
  auto kern = out_proj_tc_kernel<BN, MT>;
  AG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
  const int n_tiles_n = d / BN, n_tiles_m = (n_sub + MT - 1) / MT, n_tiles = n_tiles_n * n_tiles_m;
  kern<<<n_tiles, kThreads, Cfg::kSmemBytes, st>>>(tmO, tmW, tmY, static_cast<const __nv_bfloat16 *>(X_res), n_sub, tps,
                                                   dsc.seq, dsc.heads, d, n_tiles_m, n_tiles_n);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

// CUDA-core form: one thread per (token, output column); consecutive threads take consecutive
// columns, so the rows of W^O are read coalesced and the token's head outputs are broadcast.
template <typename T>
__global__ void __launch_bounds__(256)
out_proj_simt_kernel(const T *__restrict__ O, const T *__restrict__ Wo, const T *__restrict__ X_res, T *__restrict__ Y,
                     int n, int heads, int D, int d) {
  const int tok = blockIdx.y, c = blockIdx.x * 256 + threadIdx.x;   // tok = b n + t
  if (c >= d) return;
  const int b = tok / n, t = tok % n;
  float acc = 0.f;
  for (int i = 0; i < heads; ++i) {
    const T *o = O + (((size_t)b * heads + i) * n + t) * D;
    const T *w = Wo + (size_t)i * D * d + c;
    for (int e = 0; e < D; ++e) acc = fmaf(Elem<T>::load(o + e), Elem<T>::load(w + (size_t)e * d), acc);
  }
  if (X_res) acc += Elem<T>::load(X_res + (size_t)tok * d + c);
  Elem<T>::store(Y + (size_t)tok * d + c, acc);
}

int run_pair(const ag_layer_desc &dsc, const void *O, const void *Wo, const void *X_res, void *Y, cudaStream_t st) {
  const int d = dsc.hidden, Kdim = dsc.heads * kD;
  const int tps = (dsc.seq + kBM - 1) / kBM, n_sub = dsc.batch * tps;
  CUtensorMap tmO, tmW, tmY;
  int rc = make_tmap_3d_bf16(&tmO, O, (uint64_t)dsc.batch * dsc.heads, dsc.seq, kD, kBM, kBK);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmW, Wo, Kdim, d, (uint64_t)d * 2, kBK, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmY, Y, dsc.batch, dsc.seq, d, kBM, 64);
  if (rc) return rc;
  AG_CUDA_TRY(cudaFuncSetAttribute(out_proj_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes));
  const int n_tiles_n = d / kPairBN, n_tiles_m = (n_sub + 2 * kPairMT - 1) / (2 * kPairMT);
  out_proj_pair_kernel<<<2 * n_tiles_n * n_tiles_m, kThreads, kPairSmemBytes, st>>>(
      tmO, tmW, tmY, static_cast<const __nv_bfloat16 *>(X_res), n_sub, tps, dsc.seq, dsc.heads, d, n_tiles_m, n_tiles_n);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

template <typename T>
int run_simt(const ag_layer_desc &dsc, const void *O, const void *Wo, const void *X_res, void *Y, cudaStream_t st) {
  dim3 grid((dsc.hidden + 255) / 256, dsc.batch * dsc.seq);
  out_proj_simt_kernel<T><<<grid, 256, 0, st>>>(static_cast<const T *>(O), static_cast<const T *>(Wo),
                                                static_cast<const T *>(X_res), static_cast<T *>(Y), dsc.seq, dsc.heads,
                                                dsc.head_dim, dsc.hidden);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace

bool out_proj_tc_supported(const ag_layer_desc &d) {
  return d.dtype == AG_BF16 && d.head_dim == kD && d.hidden % 128 == 0 &&
         (int64_t)d.batch * (d.seq + kBM) < ((int64_t)1 << 31);
}

int launch_out_proj(const ag_layer_desc &d, const void *O, const void *Wo, const void *X_res, void *Y, cudaStream_t st) {
  if (out_proj_tc_supported(d)) {
    const long long tiles128 = (long long)(d.hidden / 128) * d.batch * ((d.seq + kBM - 1) / kBM);
    if (d.hidden % 256 == 0) {
      // more than one wave of 128 x 256 tiles: 512 x 256 tiles on CTA pairs, each CTA loading half of every W^O
      // stage, which keeps the tensor pipe fed from shared memory (a single CTA on a 256 x 256 tile reads 12 KB of
      // operands per MMA while TMA writes the next stage, more than shared memory's 128 B a clock)
      if (tiles128 > 2 * sm_count()) return run_pair(d, O, Wo, X_res, Y, st);
      return run_tc<256, 1>(d, O, Wo, X_res, Y, st);
    }
    return run_tc<128, 1>(d, O, Wo, X_res, Y, st);
  }
  if ((int64_t)d.batch * d.seq > 65535) return AG_ERR_UNSUPPORTED;      // grid.y of the CUDA-core form
  if (d.dtype == AG_F32) return run_simt<float>(d, O, Wo, X_res, Y, st);
  return run_simt<__nv_bfloat16>(d, O, Wo, X_res, Y, st);
}

int out_proj_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
