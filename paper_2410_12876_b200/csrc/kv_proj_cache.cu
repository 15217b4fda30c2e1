// Key/value (and, optionally, query) projection fused with selective caching: K_i = X W^K_i, V_i = X W^V_i
// (and Q_i = X W^Q_i, which goes to its dense tensor only) (Eq. 2) on the
// 5th-generation tensor cores, with an epilogue that rounds each tile to bf16 once and sends it
// to both places the layer reads it from: the dense K, V [B, h, n, D] (every token attends to its
// own key, the diagonal of Eq. 5) and, for the tokens the gate retains (Sec. 3.3: k, v are kept
// iff AG = 1), row row_off[s] + prefix[s, t] of the ragged cache.  The compaction pass over K and
// V (a read of the retained rows and a launch) disappears: the ranks prefix[s, t] are counted
// from the flags by the epilogue warps while the MMAs run.
//
// One CTA computes MT sub-tiles of 128 tokens x BN columns of the packed output [K | V]; a tile
// lies in one weight and covers BN / 128 whole heads.  Shapes whose tiles fill the SMs more than
// once run on CTA pairs (kv_proj_cache_pair_kernel).  Warp 0 drives TMA, warp 1 owns tensor
// memory and issues the MMAs, warps 2..9 drain the accumulator (two per quarter of its lanes).  Main loop as in the gate's
// projection GEMM (A = X K-major, B = W MN-major panels of [64 k][64 n], 128-byte swizzle).
// Epilogue per sub-tile: the destination rows of its tokens are computed while the MMAs run;
// the tile is staged as bf16 over the (by then free) operand stages in the layout of a swizzled
// TMA store, the dense copy leaves by TMA stores, and the retained rows are copied from the
// same staging area, one 256-byte row per half-warp.
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

namespace {

constexpr int kBM = 128, kBK = 64, kThreads = 320, kD = 128;   // warps: TMA, MMA, 8 x epilogue
constexpr int kBandTiles = 16;   // row tiles per band of the tile order

// Bytes of a 32-bit word that are not zero.
__device__ __forceinline__ int nonzero_bytes(uint32_t w) { return __popc(__vcmpne4(w, 0u) & 0x01010101u); }

template <int BN, int MT> struct KvCfg {
  static constexpr int kStages = BN == 256 ? (MT == 2 ? 3 : 4) : 6;
  static constexpr int kABytes = MT * kBM * kBK * 2;
  static constexpr int kPanelBytes = kBK * 64 * 2;           // [64 k][64 n] = 8 KB
  static constexpr int kBBytes = (BN / 64) * kPanelBytes;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kHeads = BN / kD;                     // heads per tile
  static constexpr int kDstBytes = MT * kHeads * kBM * 8;    // destination row of every (sub-tile, head, token)
  static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /*align*/ + 256 /*barriers*/ + kDstBytes + 64 /*counts*/;
};

// What the epilogue warps need besides the accumulator.
struct KvEpilogue {
  const CUtensorMap *tmK, *tmV, *tmQ;
  const uint8_t *flags;
  int32_t *prefix, *idx;
  const int64_t *row_off;
  const int32_t *cap;
  int32_t *len;
  uint8_t *k_rows, *v_rows;
  int32_t *dev_status;
  int n_sub, tps, n, kv_heads, heads;
};

// Warps 2..9 of a CTA: rank the tile's tokens while the MMAs run, then drain the CTA's mts sub-tiles
// (first sub-tile sub0, columns [nw, nw + BN) of weight `which`) from tensor memory at tmem_acc.
template <int BN, int MT>
__device__ __forceinline__ void kv_epilogue(const KvEpilogue &e, uint8_t *smem, long long *dst_row, int *red, int *gave_up,
                                            uint64_t *acc_full, uint32_t tmem_acc, int sub0, int mts, int which, int nw,
                                            int num_kb, int warp, int lane) {
  constexpr int kHeads = BN / kD;
  const uint8_t *flags = e.flags;
  int32_t *prefix = e.prefix, *idx = e.idx, *len = e.len, *dev_status = e.dev_status;
  const int64_t *row_off = e.row_off;
  const int32_t *cap = e.cap;
  const int n_sub = e.n_sub, tps = e.tps, n = e.n, kv_heads = e.kv_heads;
  const int out_heads = which == 2 ? e.heads : e.kv_heads;
  // epilogue warps: warp w may touch TMEM lanes [32 * (w % 4), +32); warps 2..5 drain the first
  // half of a sub-tile's columns, warps 6..9 the second
  const int quad = warp & 3, half = (warp - 2) >> 2;
  const int r_in = quad * 32 + lane;           // token of the sub-tile this thread drains
  // While the MMAs run: the rank of every token of the tile among the retained tokens of its slab
  // (the slab's flag row is a few KB: counted whole, as 16-byte vectors, for the number retained
  // before the tile and in the slab; the tile's own tokens ranked by warp ballot + popc), hence its
  // row in the ragged cache (-1: evicted, or the slab is too small).  The key tiles also write
  // prefix (and idx), and the one that holds a sequence's first token the slab's length.
#pragma unroll
  for (int mt = 0; mt < (half == 0 ? MT : 0); ++mt) {           // warps 2..5 only
    const int sub = sub0 + mt;
    const int b = sub / tps, t0 = (sub % tps) * kBM, t = t0 + r_in;
#pragma unroll
    for (int hh = 0; hh < kHeads; ++hh) {
      long long d = -1;
      if (sub < n_sub && mt < mts && which != 2) {                // the same for all 128 threads
        const size_t slab = (size_t)b * kv_heads + nw / kD + hh;
        const uint8_t *f = flags + slab * n;
        int before = 0, total = 0;
        if ((n & 15) == 0) {                                      // flag rows start on 16-byte boundaries
          const uint4 *fv = reinterpret_cast<const uint4 *>(f);
          for (int x = r_in; x < n / 16; x += kBM) {
            const uint4 w = ldg128(fv + x);
            const int c = nonzero_bytes(w.x) + nonzero_bytes(w.y) + nonzero_bytes(w.z) + nonzero_bytes(w.w);
            total += c;
            if (x * 16 < t0) before += c;                         // t0 is a multiple of 16: a vector lies on one side
          }
        } else {
          for (int x = r_in; x < n; x += kBM) {
            const int c = f[x] != 0;
            total += c;
            if (x < t0) before += c;
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          before += __shfl_xor_sync(0xffffffffu, before, o);
          total += __shfl_xor_sync(0xffffffffu, total, o);
        }
        const bool in_seq = t < n;                                // a single sequence may end inside its last sub-tile
        const bool keep = in_seq && f[t] != 0;
        const unsigned word = __ballot_sync(0xffffffffu, keep);
        const int in_warp = __popc(word & ((1u << lane) - 1u));
        if (lane == 0) { red[quad] = before; red[4 + quad] = total; red[8 + quad] = __popc(word); }
        named_barrier_sync(2, 128);
        before = red[0] + red[1] + red[2] + red[3];
        total = red[4] + red[5] + red[6] + red[7];
        int excl = 0;
#pragma unroll
        for (int q = 0; q < 3; ++q) excl += q < quad ? red[8 + q] : 0;
        named_barrier_sync(2, 128);                             // red is free for the next head
        const int p = before + excl + in_warp;                  // rank within the slab
        const bool fits = total <= cap[slab];
        if (fits && keep) d = row_off[slab] + p;
        if (which == 0 && in_seq) {
          int32_t *pre = prefix + slab * (n + 1);
          pre[t] = p;
          if (keep && idx) idx[slab * n + p] = t;
          if (t == 0) {
            pre[n] = total;
            len[slab] = fits ? total : 0;
            if (!fits && dev_status) atomicOr(dev_status, AG_DEV_OVERFLOW);
          }
        }
      }
      dst_row[(mt * kHeads + hh) * kBM + r_in] = d;
    }
  }
  // the eight warps start this wait at different times (warps 2..5 rank the tile's tokens first): if it
  // expires for some of them only, all of them must still agree to leave, or the barriers below would
  // wait for threads that have gone
  if (!mbar_wait(acc_full, 0)) *gave_up = 1;
  named_barrier_sync(1, 256);
  const bool ok = *gave_up == 0;
  tc_fence_after_sync();
  const CUtensorMap *tmOut = which == 0 ? e.tmK : (which == 1 ? e.tmV : e.tmQ);
  uint8_t *rows_out = which == 0 ? e.k_rows : e.v_rows;
  const int hw = (warp - 2) * 2 + (lane >> 4), l16 = lane & 15;   // half-warp 0..15, 16-byte piece of a row
#pragma unroll 1
  for (int mt = 0; mt < MT; ++mt) {
    const int sub = sub0 + mt;
    if (!ok || num_kb == 0 || sub >= n_sub || mt >= mts) break;
    const uint32_t tmem_sub = tmem_acc + mt * BN;
    // bf16 tile as panels of [128 tokens][64 columns] (128-byte rows, 16-byte chunks XOR-swizzled by the
    // row); each sub-tile has a staging area of its own, so the second is drained while the first leaves
    uint8_t *stg = smem + mt * (BN / 64) * kBM * 128;
#pragma unroll 1
    for (int c = half * (BN / 2); c < (half + 1) * (BN / 2); c += 32) {
      uint32_t r[32];
      tmem_ld_x32_sync(tmem_sub + ((uint32_t)(quad * 32) << 16) + c, r);
      const uint32_t panel = (uint32_t)(c >> 6) * kBM * 128 + r_in * 128;
#pragma unroll
      for (int e = 0; e < 32; e += 8) {
        uint32_t h[4];
#pragma unroll
        for (int q = 0; q < 8; q += 2)
          h[q >> 1] = pack_bf16x2(__uint_as_float(r[e + q]), __uint_as_float(r[e + q + 1]));
        const uint32_t chunk = (uint32_t)(((c & 32) >> 3) + (e >> 3));
        *reinterpret_cast<uint4 *>(stg + panel + ((chunk ^ (r_in & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
      }
    }
    fence_proxy_async_smem();
    named_barrier_sync(1, 256);                  // the tile is staged (and dst_row written, first time round)
    const int b = sub / tps, t0 = (sub % tps) * kBM;
    if (threadIdx.x == 64) {
#pragma unroll
      for (int p = 0; p < BN / 64; ++p)
        tma_store_3d(tmOut, stg + p * kBM * 128, (p & 1) * 64, t0, b * out_heads + nw / kD + (p >> 1));
      tma_store_commit();
    }
    // retained rows: half-warp per row, 16 bytes per lane
#pragma unroll
    for (int hh = 0; hh < (which != 2 ? kHeads : 0); ++hh) {
      const long long *dr = dst_row + (mt * kHeads + hh) * kBM;
#pragma unroll 4
      for (int r = hw; r < kBM; r += 16) {
        const long long d = dr[r];
        if (d >= 0) {
          const uint32_t off = (uint32_t)(hh * 2 + (l16 >> 3)) * kBM * 128 + r * 128 + (((l16 & 7) ^ (r & 7)) << 4);
          *reinterpret_cast<uint4 *>(rows_out + (size_t)d * (kD * 2) + l16 * 16) =
              *reinterpret_cast<const uint4 *>(stg + off);
        }
      }
    }
  }
  if (threadIdx.x == 64) tma_store_wait_read();
}

template <int BN, int MT>
__global__ void __launch_bounds__(kThreads, 1)
kv_proj_cache_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBk,
                     const __grid_constant__ CUtensorMap tmBv, const __grid_constant__ CUtensorMap tmBq,
                     const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                     const __grid_constant__ CUtensorMap tmQ, const uint8_t *__restrict__ flags,
                     int32_t *__restrict__ prefix, int32_t *__restrict__ idx, const int64_t *__restrict__ row_off,
                     const int32_t *__restrict__ cap, int32_t *__restrict__ len, uint8_t *__restrict__ k_rows,
                     uint8_t *__restrict__ v_rows, int32_t *__restrict__ dev_status, int n_sub, int tps, int Kdim, int GD,
                     int n, int kv_heads, int heads, int n_tiles_m, int n_tiles_n) {
  using Cfg = KvCfg<BN, MT>;
  constexpr uint32_t kTmemCols = MT * BN;
  static_assert(kTmemCols == 128 || kTmemCols == 256 || kTmemCols == 512, "TMEM columns: a power of two");
  static_assert(MT * (BN / 64) * kBM * 128 <= Cfg::kStages * Cfg::kStageBytes, "staging fits the stages");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + Cfg::kStages * Cfg::kStageBytes);
  uint64_t *empty = full + Cfg::kStages;
  uint64_t *acc_full = empty + Cfg::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  long long *dst_row = reinterpret_cast<long long *>(smem + Cfg::kStages * Cfg::kStageBytes + 256);
  int *red = reinterpret_cast<int *>(smem + Cfg::kStages * Cfg::kStageBytes + 256 + Cfg::kDstBytes);   // 12 ints
  int *gave_up = red + 12;                       // set by an epilogue thread whose wait for the accumulator expired

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x;
  // tile order: bands of kBandTiles row tiles; inside a band the row tile runs fastest, so the CTAs in
  // flight share a few column slices of W while the band's rows of X stay in L2
  const int band = tile / (kBandTiles * n_tiles_n), in_band = tile % (kBandTiles * n_tiles_n);
  const int band_rows = min(kBandTiles, n_tiles_m - band * kBandTiles);
  const int tile_m = band * kBandTiles + in_band % band_rows, tile_n = in_band / band_rows;
  // Rows are counted in sub-tiles of 128 tokens laid out per sequence: sequence b owns sub-tiles
  // [b tps, (b + 1) tps), the last of which may reach past the sequence's end (those rows are zeros on
  // the way in, take no rank, and are dropped by the stores), so a sub-tile never spans two sequences.
  const int sub0 = tile_m * MT;
  const int n0 = tile_n * BN;                    // in the packed output [K | V | Q] (GD, GD and heads * D columns)
  // BN divides the width of every weight: a tile lies in one weight.  which: 0 keys, 1 values, 2 queries
  // (queries go to their dense tensor only: no flags, no cache)
  const int which = n0 < GD ? 0 : (n0 < 2 * GD ? 1 : 2);
  const int nw = n0 - min(which, 2) * GD;
  const CUtensorMap *tmB = which == 0 ? &tmBk : (which == 1 ? &tmBv : &tmBq);
  const int num_kb = (Kdim + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(tmB);
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
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)              // rows past the sequence (or past the batch) are filled with zeros
          tma_load_3d(a + mt * (kBM * kBK * 2), &tmA, &full[s], kb * kBK, ((sub0 + mt) % tps) * kBM, (sub0 + mt) / tps);
#pragma unroll
        for (int p = 0; p < BN / 64; ++p)
          tma_load_2d(b + p * Cfg::kPanelBytes, tmB, &full[s], nw + p * 64, kb * kBK);
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
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % Cfg::kStages;
      const uint32_t ph = (kb / Cfg::kStages) & 1;
      ok = mbar_wait(&full[s], ph);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t a_lo = a_lo0 + ((s * Cfg::kStageBytes) >> 4), b_lo = b_lo0 + ((s * Cfg::kStageBytes) >> 4);
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt)
            mma_ss_lohi(tmem_acc + mt * BN, a_lo + ((mt * kBM * kBK * 2 + k * 32) >> 4), a_hi,
                        b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
        }
        mma_commit(&empty[s]);     // frees the stage once these MMAs have read it
      }
      __syncwarp();
    }
    if (elect_one()) mma_commit(acc_full);   // accumulator complete (or unwinding)
    __syncwarp();
  } else {
    const KvEpilogue e{&tmK, &tmV, &tmQ, flags, prefix, idx, row_off, cap, len, k_rows, v_rows, dev_status, n_sub, tps, n, kv_heads, heads};
    kv_epilogue<BN, MT>(e, smem, dst_row, red, gave_up, acc_full, tmem_acc, sub0, MT, which, nw, num_kb, warp, lane);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// The same projection on CTA pairs (cta_group::2): a pair computes 512 tokens x 256 columns, each CTA
// holding its own two sub-tiles of X and half of every stage of W, the leader issuing M = 256 MMAs
// whose accumulators land in both CTAs' tensor memory.  A single CTA on a 256 x 256 tile reads 12 KB
// of operands from shared memory per MMA while TMA writes the next stage, more than shared memory
// moves in the MMA's 128 clocks; here it is 8 KB.  The pair tiles of a last wave that would fill at
// most half of the SMs go to two pairs of 256 tokens each.
constexpr int kPairBN = 256, kPairMT = 2, kPairStages = 4;
constexpr int kPairABytes = kPairMT * kBM * kBK * 2;                 // 32 KB: this CTA's two sub-tiles of X
constexpr int kPairBBytes = (kPairBN / 2 / 64) * (kBK * 64 * 2);     // 16 KB: this CTA's half of the stage of W
constexpr int kPairBandTiles = 8;   // pair tiles of rows per band: the same 4096 tokens of A as a band of single-CTA tiles
constexpr int kPairStageBytes = kPairABytes + kPairBBytes;           // 48 KB
constexpr int kPairDstBytes = kPairMT * (kPairBN / kD) * kBM * 8;
constexpr int kPairSmemBytes = kPairStages * kPairStageBytes + 1024 + 256 + kPairDstBytes + 64;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
kv_proj_cache_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBk,
                          const __grid_constant__ CUtensorMap tmBv, const __grid_constant__ CUtensorMap tmBq,
                          const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                          const __grid_constant__ CUtensorMap tmQ, const uint8_t *__restrict__ flags,
                          int32_t *__restrict__ prefix, int32_t *__restrict__ idx, const int64_t *__restrict__ row_off,
                          const int32_t *__restrict__ cap, int32_t *__restrict__ len, uint8_t *__restrict__ k_rows,
                          uint8_t *__restrict__ v_rows, int32_t *__restrict__ dev_status, int n_sub, int tps, int Kdim,
                          int GD, int n, int kv_heads, int heads, int n_tiles_m, int n_tiles_n, int split_from) {
  constexpr int BN = kPairBN, MT = kPairMT;
  constexpr uint32_t kTmemCols = MT * BN;          // 512: two accumulators of 128 rows x 256 columns per CTA
  static_assert(MT * (BN / 64) * kBM * 128 <= kPairStages * kPairStageBytes, "staging fits the stages");
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kPairStages * kPairStageBytes);   // used in the leader only
  uint64_t *empty = full + kPairStages;            // one set per CTA: a commit arrives on both
  uint64_t *acc_full = empty + kPairStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
  long long *dst_row = reinterpret_cast<long long *>(smem + kPairStages * kPairStageBytes + 256);
  int *red = reinterpret_cast<int *>(smem + kPairStages * kPairStageBytes + 256 + kPairDstBytes);
  int *gave_up = red + 12;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();         // 0: leader
  // pairs below split_from take whole pair tiles, the rest one half (256 tokens) of a pair tile
  const int pair = blockIdx.x >> 1;
  const bool single = pair >= split_from;
  const int tile = single ? split_from + ((pair - split_from) >> 1) : pair;
  const int mts = single ? 1 : MT;                 // sub-tiles of each CTA
  const int band = tile / (kPairBandTiles * n_tiles_n), in_band = tile % (kPairBandTiles * n_tiles_n);
  const int band_rows = min(kPairBandTiles, n_tiles_m - band * kPairBandTiles);
  const int tile_m = band * kPairBandTiles + in_band % band_rows, tile_n = in_band / band_rows;
  const int sub0 = tile_m * (2 * MT) + (single ? ((pair - split_from) & 1) * 2 + (int)rank : (int)rank * MT);
  const int n0 = tile_n * BN;
  const int which = n0 < GD ? 0 : (n0 < 2 * GD ? 1 : 2);
  const int nw = n0 - min(which, 2) * GD;
  const CUtensorMap *tmB = which == 0 ? &tmBk : (which == 1 ? &tmBv : &tmBq);
  const int num_kb = (Kdim + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    *gave_up = 0;
    fence_barrier_init();
    prefetch_tensormap(&tmA);
    prefetch_tensormap(tmB);
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
  const uint32_t stage_tx = (uint32_t)(mts * (kBM * kBK * 2) + kPairBBytes);

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kPairStages;
        const uint32_t ph = (kb / kPairStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1)) break;  // this CTA's copy: the MMAs that read the stage (in both CTAs) are done
        uint8_t *a = smem + s * kPairStageBytes, *b = a + kPairABytes;
        if (rank == 0) mbar_arrive_expect_tx(&full[s], 2 * stage_tx);   // the leader's barrier counts both CTAs' bytes
        const uint32_t bar = mapa_shared(smem_u32(&full[s]), 0);
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)            // rows past the sequence (or past the batch) are filled with zeros
          if (mt < mts)
            tma_load_3d_pair(a + mt * (kBM * kBK * 2), &tmA, bar, kb * kBK, ((sub0 + mt) % tps) * kBM, (sub0 + mt) / tps);
#pragma unroll
        for (int p = 0; p < BN / 2 / 64; ++p)      // this CTA's half of the tile's columns
          tma_load_2d_pair(b + p * (kBK * 64 * 2), tmB, bar, nw + (int)rank * (BN / 2) + p * 64, kb * kBK);
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
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % kPairStages;
        const uint32_t ph = (kb / kPairStages) & 1;
        ok = mbar_wait(&full[s], ph);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a_lo = a_lo0 + ((s * kPairStageBytes) >> 4), b_lo = b_lo0 + ((s * kPairStageBytes) >> 4);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
              if (mt < mts) mma_ss_pair_lohi(tmem_acc + mt * BN, a_lo + ((mt * kBM * kBK * 2 + k * 32) >> 4), a_hi,
                                             b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
          }
          mma_commit_pair(&empty[s]);              // frees the stage in both CTAs once these MMAs have read it
        }
        __syncwarp();
      }
      if (elect_one()) mma_commit_pair(acc_full);  // accumulators complete (or unwinding), in both CTAs
      __syncwarp();
    }
  } else {
    const KvEpilogue e{&tmK, &tmV, &tmQ, flags, prefix, idx, row_off, cap, len, k_rows, v_rows, dev_status, n_sub, tps, n, kv_heads, heads};
    kv_epilogue<BN, MT>(e, smem, dst_row, red, gave_up, acc_full, tmem_acc, sub0, mts, which, nw, num_kb, warp, lane);
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
int run(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk, const void *Wv, const uint8_t *flags,
        const ag_cache &c, int32_t *prefix, int32_t *idx, void *Q, void *K, void *V, int32_t *dev_status,
        cudaStream_t st, bool pairs = false) {
  using Cfg = KvCfg<BN, MT>;
  const int hk = kv_heads_of(d), GD = hk * kD, Kdim = d.hidden;
  const int tps = (d.seq + kBM - 1) / kBM, n_sub = d.batch * tps;   // sub-tiles of 128 tokens per sequence, in all
  const int QD = Wq ? d.heads * kD : 0;          // query columns of the packed output (0: keys and values only)
  CUtensorMap tmA, tmBk, tmBv, tmBq, tmK, tmV, tmQ;
  int rc = make_tmap_3d_bf16(&tmA, X, d.batch, d.seq, Kdim, kBM, kBK);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmBk, Wk, Kdim, GD, (uint64_t)GD * 2, kBK, 64);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmBv, Wv, Kdim, GD, (uint64_t)GD * 2, kBK, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmK, K, (uint64_t)d.batch * hk, d.seq, kD, kBM, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmV, V, (uint64_t)d.batch * hk, d.seq, kD, kBM, 64);
  if (rc) return rc;
  tmBq = tmBk;                                   // stand-ins when there is no query projection
  tmQ = tmK;
  if (Wq) {
    rc = make_tmap_2d_bf16(&tmBq, Wq, Kdim, QD, (uint64_t)QD * 2, kBK, 64);
    if (rc) return rc;
    rc = make_tmap_3d_bf16(&tmQ, Q, (uint64_t)d.batch * d.heads, d.seq, kD, kBM, 64);
    if (rc) return rc;
  }
  if (pairs) {
    // 512 x 256 tiles on CTA pairs; the tiles of a last wave that would fill at most half of the pairs are halved
    AG_CUDA_TRY(cudaFuncSetAttribute(kv_proj_cache_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes));
    const int n_tiles_n = (2 * GD + QD) / kPairBN, n_tiles_m = (n_sub + 2 * kPairMT - 1) / (2 * kPairMT);
    const int n_tiles = n_tiles_n * n_tiles_m, n_pairs = sm_count() / 2;
    const int tail = n_tiles % n_pairs;
    const int split_from = (tail > 0 && 2 * tail <= n_pairs) ? n_tiles - tail : n_tiles;
    const int ctas = 2 * (split_from + 2 * (n_tiles - split_from));
    kv_proj_cache_pair_kernel<<<ctas, kThreads, kPairSmemBytes, st>>>(
        tmA, tmBk, tmBv, tmBq, tmK, tmV, tmQ, flags, prefix, idx, c.row_off, c.cap, c.len, static_cast<uint8_t *>(c.k_rows),
        static_cast<uint8_t *>(c.v_rows), dev_status, n_sub, tps, Kdim, GD, d.seq, hk, d.heads, n_tiles_m, n_tiles_n, split_from);
    AG_LAUNCH_CHECK();
    return AG_OK;
  }
  auto kern = kv_proj_cache_kernel<BN, MT>;
  AG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes));
  const int n_tiles_n = (2 * GD + QD) / BN, n_tiles_m = (n_sub + MT - 1) / MT, n_tiles = n_tiles_n * n_tiles_m;
  kern<<<n_tiles, kThreads, Cfg::kSmemBytes, st>>>(tmA, tmBk, tmBv, tmBq, tmK, tmV, tmQ, flags, prefix, idx, c.row_off, c.cap, c.len,
                                                   static_cast<uint8_t *>(c.k_rows), static_cast<uint8_t *>(c.v_rows),
                                                   dev_status, n_sub, tps, Kdim, GD, d.seq, hk, d.heads, n_tiles_m, n_tiles_n);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace

bool kv_proj_cache_supported(const ag_layer_desc &d) {
  return d.dtype == AG_BF16 && d.head_dim == kD && d.hidden > 0 && d.hidden % 8 == 0 &&
         (int64_t)d.batch * (d.seq + kBM) < ((int64_t)1 << 31);
}

int launch_kv_proj_cache(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk, const void *Wv,
                         const uint8_t *flags, const ag_cache &c, int32_t *prefix, int32_t *idx, void *Q, void *K,
                         void *V, int32_t *dev_status, cudaStream_t st) {
  const int hk = kv_heads_of(d), hq = Wq ? d.heads : 0;
  const long long tiles128 = (long long)(2 * hk + hq) * d.batch * ((d.seq + kBM - 1) / kBM);
  int rc;
  if (hk % 2 == 0 && hq % 2 == 0) {
    // more than one wave: CTA pairs on 512 x 256 tiles
    if (tiles128 > 2 * sm_count()) rc = run<256, 1>(d, X, Wq, Wk, Wv, flags, c, prefix, idx, Q, K, V, dev_status, st, true);
    else rc = run<256, 1>(d, X, Wq, Wk, Wv, flags, c, prefix, idx, Q, K, V, dev_status, st);
  } else {
    rc = run<128, 1>(d, X, Wq, Wk, Wv, flags, c, prefix, idx, Q, K, V, dev_status, st);
  }
  if (rc) return rc;
  // recent-token window: the ring takes the prompt's last tokens from the dense K, V just written
  return launch_recent_fill(d, K, V, flags, c, st);
}

int kv_proj_cache_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
