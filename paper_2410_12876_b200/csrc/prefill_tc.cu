// Prefill attention under the eviction mask (Eq. 2 with M_i of Eq. 5) on the
// Blackwell tensor cores, bf16, head_dim 128.
//
// One CTA handles 128 consecutive queries of one slab s = (sequence, head).
// Query j attends to cache rows r < prefix[s, j] (exactly the retained tokens
// before j, Sec. 3.3) and to itself (the diagonal of Eq. 5, always kept).  Over
// the compacted rows the mask is a staircase, so only the tiles that touch it
// need per-element masking and evicted keys are never loaded.
//
//   warp 0      TMA: Q tile once, then K / V tiles of 64 cache rows (2 stages)
//   warp 1      owns tensor memory, issues S = Q K^T (tcgen05.mma, operands in
//               shared memory) and O += P V (P read from tensor memory)
//   warps 2..5  one query row per thread: online softmax on S read from TMEM,
//               P written back to TMEM as bf16, O rescaled only when the running
//               maximum grows by more than 2^8, final normalisation and store
//
// TMEM columns: S0 [0,64) S1 [64,128), each overwritten in place by its P (bf16 pairs); O [128,256).
// The self term seeds the running softmax (m = s_jj, l = 1) and its value row
// is added in the epilogue: O_j = (sum_r p_r v_r + w_self v_j) / l.  Every byte
// that enters or leaves the CTA travels by TMA.
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

constexpr int kPfThreads = 192;
constexpr int kPfBM = 128, kPfD = 128;
constexpr int kPfPanel = 128 * 128;                   // [128 rows][64 bf16] = 16 KB (Q, dense K / V, O)
constexpr int kPfTile = 2 * kPfPanel;                 // 32 KB
constexpr float kRescaleThreshold = 8.f;              // log2 units

// Key tiles of 64 cache rows; two CTAs per SM (256 TMEM columns, 97 KB of shared memory each).
// 128-row tiles with one CTA per SM measured slower on 4096-token heads (131 us against 100 us).
constexpr int kPfBN = 64;
constexpr int kPfKvPanel = kPfBN * 128;               // [64 rows][64 bf16] = 8 KB
constexpr int kPfKvTile = 2 * kPfKvPanel;             // 16 KB
constexpr int kPfKvBuf = 2 * kPfKvTile;               // two stages = one 32 KB dense tile
constexpr int kPfSmemBytes = kPfTile + 2 * kPfKvBuf + 1024 + 256;
constexpr uint32_t kColS = 0, kColO = 2 * kPfBN, kTmemCols = 256;
constexpr int kPfCtasPerSm = 2;

struct PrefillTcArgs {
  const int32_t *prefix;            // [slabs, n + 1]
  const int64_t *row_off;
  const int32_t *len;
  int n, n_qtiles, slabs;           // slabs: (sequence, query head) pairs
  int heads, kv_heads;              // query heads share key/value heads in groups of heads / kv_heads
  float scale_log2;
  float *lse;                       // NULL, or [slabs, n]: m + log2(l) of every row (see launch_prefill_tc)
  const int32_t *seq_lens;          // NULL, or [batch]: a query tile that holds padding only is skipped
};

// Byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a [128 x 128] bf16 tile stored
// as two 128-byte-swizzled panels of 64 columns (the layout TMA writes and tcgen05.mma reads).
__device__ __forceinline__ uint32_t tile_chunk_offset(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * kPfPanel + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}

// Two CTAs share an SM (256 TMEM columns, 97 KB of shared memory each).  Keys
// are visited in tiles of 64 with S double-buffered, so S = Q K^T of tile i + 1
// runs while the softmax threads work on tile i and O += P V of tile i runs
// while they work on tile i + 1: the softmax threads never wait for the tensor
// core in steady state, and the tensor core interleaves the two CTAs.
//
// The first MMA tile is the "self tile": S = Q_tile Kdense_tile^T over the
// CTA's own 128 rows, of which only the diagonal (q_j . k_j) is read.  Last,
// the dense V tile is brought in for the self term of the output, and the O
// tile leaves through shared memory with one TMA store.
__global__ void __launch_bounds__(kPfThreads, kPfCtasPerSm)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKd,
                  const __grid_constant__ CUtensorMap tmVd, const __grid_constant__ CUtensorMap tmO,
                  const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                  const PrefillTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;
  uint8_t *sK = sQ + kPfTile;                      // two stages, or one 128-row dense tile
  uint8_t *sV = sK + kPfKvBuf;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sV + kPfKvBuf);
  uint64_t *q_full = bars;
  uint64_t *k_full = bars + 1, *k_empty = bars + 3, *v_full = bars + 5, *v_empty = bars + 7;   // [2] each
  uint64_t *s_full = bars + 9;                     // [2]
  // p_ready[2], pv_done[2]: even / odd cache tiles.  Two p_ready barriers because a softmax warp
  // may finish tile i + 1 before a slower one has finished tile i; it cannot get further ahead,
  // since S of tile i + 2 waits for the P V of tile i.
  uint64_t *p_ready = bars + 11, *pv_done = bars + 13, *self_full = bars + 15;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 16);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // heaviest query tiles first
  const int qt = a.n_qtiles - 1 - (int)(blockIdx.x / a.slabs);
  const int slab = blockIdx.x % a.slabs;           // Q and O live here
  // a query tile past its sequence's end holds padding only: its outputs are unspecified, nothing to do
  if (a.seq_lens != nullptr && qt * kPfBM >= a.seq_lens[slab / a.heads]) return;
  // K, V, the flags' prefix counts and the cache belong to the key/value head (grouped-query attention)
  const int kv_slab = (slab / a.heads) * a.kv_heads + (slab % a.heads) / (a.heads / a.kv_heads);
  const int j0 = qt * kPfBM;
  const int j_last = min(j0 + kPfBM, a.n) - 1;
  const int32_t *pre = a.prefix + (size_t)kv_slab * (a.n + 1);
  // keys any row of this tile may see; never past the slab's valid rows (a slab that overflowed at
  // compaction has len = 0 under full prefix counts: its queries see themselves only)
  const int max_bound = min(pre[j_last], a.len[kv_slab]);
  const int n_kv = (max_bound + kPfBN - 1) / kPfBN;
  const int row0 = (int)a.row_off[kv_slab];
  static_assert(kPfKvBuf == kPfTile, "the self tile below spans exactly the two V stages");
  // uses of K stage 0 / 1 before the dense V tile: even / odd cache tiles
  const int k0_uses = (n_kv + 1) / 2, k1_uses = n_kv / 2;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
      mbar_init(&s_full[s], 1);
    }
    mbar_init(&p_ready[0], 128); mbar_init(&p_ready[1], 128);
    mbar_init(&pv_done[0], 1); mbar_init(&pv_done[1], 1);
    mbar_init(self_full, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmQ); prefetch_tensormap(&tmKd); prefetch_tensormap(&tmVd);
    prefetch_tensormap(&tmK); prefetch_tensormap(&tmV); prefetch_tensormap(&tmO);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      bool ok = true;
      if (n_kv > 0) {
        mbar_arrive_expect_tx(q_full, kPfTile);
        tma_load_3d(sQ, &tmQ, q_full, 0, j0, slab);
        tma_load_3d(sQ + kPfPanel, &tmQ, q_full, 64, j0, slab);
        // self tile: dense K rows j0 .. j0 + 127 across both V stages, which no P V needs before
        // the first softmax is done; the first cache tiles of K load alongside it
        mbar_arrive_expect_tx(&v_full[0], kPfTile);
        tma_load_3d(sV, &tmKd, &v_full[0], 0, j0, kv_slab);
        tma_load_3d(sV + kPfPanel, &tmKd, &v_full[0], 64, j0, kv_slab);
        for (int i = 0; i < n_kv && ok; ++i) {
          const int st = i & 1;
          const int y = row0 + i * kPfBN;
          ok = mbar_wait(&k_empty[st], ((i >> 1) & 1) ^ 1);     // earlier uses of the stage: i >> 1
          if (!ok) break;
          mbar_arrive_expect_tx(&k_full[st], kPfKvTile);
          tma_load_2d(sK + st * kPfKvTile, &tmK, &k_full[st], 0, y);
          tma_load_2d(sK + st * kPfKvTile + kPfKvPanel, &tmK, &k_full[st], 64, y);
          ok = mbar_wait(&v_empty[st], (i >> 1) & 1);           // the self tile + i >> 1 earlier tiles
          if (!ok) break;
          mbar_arrive_expect_tx(&v_full[st], kPfKvTile);
          tma_load_2d(sV + st * kPfKvTile, &tmV, &v_full[st], 0, y);
          tma_load_2d(sV + st * kPfKvTile + kPfKvPanel, &tmV, &v_full[st], 64, y);
        }
      }
      // dense V rows for the self term of the output, into the K buffer once both stages are free
      if (ok && k0_uses > 0) ok = mbar_wait(&k_empty[0], (k0_uses & 1) ^ 1);
      if (ok && k1_uses > 0) ok = mbar_wait(&k_empty[1], (k1_uses & 1) ^ 1);
      if (ok) {
        mbar_arrive_expect_tx(&k_full[0], kPfTile);
        tma_load_3d(sK, &tmVd, &k_full[0], 0, j0, kv_slab);
        tma_load_3d(sK + kPfPanel, &tmVd, &k_full[0], 64, j0, kv_slab);
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    // Every lane runs the control flow so that operands stay warp-uniform (the tensor-core
    // instructions take uniform registers); one elected lane issues.
    if (n_kv > 0) {
      // descriptors as (low, high) words: the high words are fixed per operand kind, the low
      // words are a base plus a compile-time offset per K step
      const uint64_t dq = desc_kmajor_sw128(smem_u32(sQ)), dk = desc_kmajor_sw128(smem_u32(sK));
      const uint64_t dself = desc_kmajor_sw128(smem_u32(sV));
      const uint64_t dv = desc_mnmajor_sw128(smem_u32(sV), kPfKvPanel);
      const uint32_t q_lo = (uint32_t)dq, q_hi = (uint32_t)(dq >> 32);
      const uint32_t k_lo = (uint32_t)dk, k_hi = (uint32_t)(dk >> 32);
      const uint32_t v_lo = (uint32_t)dv, v_hi = (uint32_t)(dv >> 32);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(kPfBM, kPfD, false, true);
      // keys of cache tile i any row can see, rounded up to the MMA's N / K granularity
      auto tile_keys = [&](int i) { return min(kPfBN, (max_bound - i * kPfBN + 15) & ~15); };
      auto issue_qk = [&](int i) -> bool {
        const int st = i & 1;
        if (!mbar_wait(&k_full[st], (i >> 1) & 1)) return false;
        tc_fence_after_sync();
        const uint32_t idesc_qk = idesc_bf16_f32(kPfBM, tile_keys(i), false, false);
        const uint32_t kb = k_lo + ((st * kPfKvTile) >> 4);
        const uint32_t d = tmem + kColS + st * kPfBN;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kPfD / 16; ++k)
            mma_ss_lohi(d, q_lo + (((k >> 2) * kPfPanel + (k & 3) * 32) >> 4), q_hi,
                        kb + (((k >> 2) * kPfKvPanel + (k & 3) * 32) >> 4), k_hi, idesc_qk, k != 0);
          mma_commit(&k_empty[st]);
          mma_commit(&s_full[st]);
        }
        __syncwarp();
        return true;
      };
      bool ok = mbar_wait(q_full, 0);
      // self tile: 128 dense K rows (in the V stages); its scores land in the columns of O,
      // which are free until the first P V - that one starts a fresh accumulation, and it cannot
      // be issued before the softmax threads, who read the diagonal first, are done with tile 0
      ok = ok && mbar_wait(&v_full[0], 0);
      if (ok) {
        tc_fence_after_sync();
        constexpr uint32_t idesc_self = idesc_bf16_f32(kPfBM, 128, false, false);
        const uint32_t s_lo = (uint32_t)dself, s_hi = (uint32_t)(dself >> 32);
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kPfD / 16; ++k) {
            const uint32_t off = ((k >> 2) * kPfPanel + (k & 3) * 32) >> 4;
            mma_ss_lohi(tmem + kColO, q_lo + off, q_hi, s_lo + off, s_hi, idesc_self, k != 0);
          }
          mma_commit(&v_empty[0]);
          mma_commit(&v_empty[1]);
          mma_commit(self_full);
        }
        __syncwarp();
      }
      ok = ok && issue_qk(0);
      for (int i = 0; i < n_kv && ok; ++i) {
        if (i + 1 < n_kv) {
          // S[(i+1)&1] still holds P of tile i - 1 until that P V has completed
          if (i >= 1 && !mbar_wait(&pv_done[(i - 1) & 1], ((i - 1) >> 1) & 1)) { ok = false; break; }
          if (!issue_qk(i + 1)) { ok = false; break; }
        }
        const int st = i & 1;
        if (!mbar_wait(&p_ready[st], (i >> 1) & 1)) { ok = false; break; }
        // V stage 0 has held the self tile before (stage 1 shared that load's barrier)
        if (!mbar_wait(&v_full[st], ((i >> 1) + (st == 0 ? 1 : 0)) & 1)) { ok = false; break; }
        tc_fence_after_sync();
        const int ksteps = tile_keys(i) / 16;
        const uint32_t vb = v_lo + ((st * kPfKvTile) >> 4);
        const uint32_t pa = tmem + kColS + st * kPfBN;
        if (elect_one()) {
#pragma unroll
          for (int k = 0; k < kPfBN / 16; ++k)
            if (k < ksteps) mma_ts_lohi(tmem + kColO, pa + k * 8, vb + ((k * 2048) >> 4), v_hi, idesc_pv, (i | k) != 0);
          mma_commit(&v_empty[st]);
          mma_commit(&pv_done[st]);
        }
        __syncwarp();
      }
    }
  } else {
    // ------------------------------------------- softmax / correction / epilogue
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;
    const int tid = threadIdx.x - 64;                // 0..127
    const int j = j0 + row;
    const bool valid = j < a.n;
    const int L = a.len[kv_slab];
    const int bound = valid ? min(pre[j], L) : 0;
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    float m = 0.f, self2 = 0.f, l = 1.f;
    bool ok = true;

    if (n_kv > 0) {
      // self tile: this thread's diagonal element S[row][row] = q_j . k_j
      ok = mbar_wait(self_full, 0);
      tc_fence_after_sync();
      uint32_t d[32];
      tmem_ld_x32_sync(tm_lane + kColO + quad * 32, d);
      float s_self = 0.f;
#pragma unroll
      for (int e = 0; e < 32; ++e) s_self = (e == lane) ? __uint_as_float(d[e]) : s_self;
      self2 = s_self * a.scale_log2;
      m = self2;
    }

    for (int i = 0; i < n_kv && ok; ++i) {
      const int st = i & 1;
      ok = mbar_wait(&s_full[st], (i >> 1) & 1);
      if (!ok) break;
      tc_fence_after_sync();
      const int nvalid = min(max(bound - i * kPfBN, 0), kPfBN);
      const uint32_t tS = tm_lane + kColS + st * kPfBN;

      uint32_t r[kPfBN];
      tmem_ld_x64_sync(tS, r);
      if (nvalid < kPfBN) {
#pragma unroll
        for (int e = 0; e < kPfBN; ++e)
          if (e >= nvalid) r[e] = 0xff800000u;        // -inf: weight 0 below
      }
      // eight independent chains instead of one long dependency, two elements per instruction
      float mx[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) mx[q] = max3_f32(__uint_as_float(r[q]), __uint_as_float(r[q + 8]), __uint_as_float(r[q + 16]));
#pragma unroll
      for (int e = 24; e + 8 < kPfBN; e += 16)
#pragma unroll
        for (int q = 0; q < 8; ++q) mx[q] = max3_f32(mx[q], __uint_as_float(r[e + q]), __uint_as_float(r[e + q + 8]));
#pragma unroll
      for (int q = 0; q < 8; ++q) mx[q] = fmaxf(mx[q], __uint_as_float(r[kPfBN - 8 + q]));
      float tmax = max3_f32(max3_f32(mx[0], mx[1], mx[2]), max3_f32(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]));
      tmax *= a.scale_log2;                           // scale > 0: max commutes; -inf stays -inf
      float m_new;
      if (i == 0) m_new = fmaxf(m, tmax);
      else m_new = (tmax > m + kRescaleThreshold) ? tmax : m;
      const bool rescale = (i > 0) && __any_sync(0xffffffffu, m_new != m);
      const float alpha = fast_exp2(m - m_new);

      // p = 2^(s - m) as bf16 pairs, written over the columns S occupied; the scaling and the row
      // sums two elements per instruction
      float rs[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      const float neg_m = -m_new;
#pragma unroll
      for (int c = 0; c < kPfBN / 16; ++c) {
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          float t0, t1;
          fma_f32x2(t0, t1, __uint_as_float(r[c * 16 + e]), __uint_as_float(r[c * 16 + e + 1]), a.scale_log2,
                    a.scale_log2, neg_m, neg_m);
          const float p0 = fast_exp2(t0), p1 = fast_exp2(t1);
          const int k = ((e >> 1) & 3) * 2;
          add_f32x2(rs[k], rs[k + 1], rs[k], rs[k + 1], p0, p1);
          pk[e >> 1] = pack_bf16x2(p0, p1);
        }
        tmem_st_x8(tS + c * 8, pk);
      }
      l = l * alpha + (((rs[0] + rs[1]) + (rs[2] + rs[3])) + ((rs[4] + rs[5]) + (rs[6] + rs[7])));
      m = m_new;

      // Only a rescale of O has to wait for the P V of tile i - 1.  The parity wait is unambiguous
      // although this thread has not watched every phase of that barrier: the P V of tile i - 3
      // (the barrier's previous phase) completed before the Q K^T of tile i - 1 was issued, whose
      // scores this thread has already used, and the P V of tile i + 1 cannot have been issued yet.
      if (rescale) {
        ok = mbar_wait(&pv_done[(i - 1) & 1], ((i - 1) >> 1) & 1);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_x32_sync(tm_lane + kColO + c * 32, o);
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st_x32(tm_lane + kColO + c * 32, o);
        }
      }

      // Rows of the V tile past the slab's valid length hold whatever the pool
      // holds (possibly NaN bit patterns): their weight is 0, but 0 * NaN is NaN
      // in the tensor core, so zero them in shared memory before P V reads them.
      if ((i + 1) * kPfBN > L) {
        ok = mbar_wait(&v_full[st], ((i >> 1) + (st == 0 ? 1 : 0)) & 1);
        if (!ok) break;
        const int vr = tid >> 1;                      // two threads per row, one panel each
        if (i * kPfBN + vr >= L) {
          uint4 z = make_uint4(0, 0, 0, 0);
          uint8_t *v0 = sV + st * kPfKvTile + (tid & 1) * kPfKvPanel + vr * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4 *>(v0 + c * 16) = z;
        }
        fence_proxy_async_smem();
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&p_ready[st]);
    }

    // epilogue: O_j = (sum_r p_r v_r + w_self v_j) / l, staged in the V buffer, one TMA store
    if (ok && n_kv > 1) ok = mbar_wait(&pv_done[(n_kv - 2) & 1], ((n_kv - 2) >> 1) & 1);
    if (ok && n_kv > 0) {
      ok = mbar_wait(&pv_done[(n_kv - 1) & 1], ((n_kv - 1) >> 1) & 1);
      tc_fence_after_sync();
    }
    if (ok) ok = mbar_wait(&k_full[0], k0_uses & 1);          // dense V tile has landed in sK
    if (ok) {
      const float w_self = fast_exp2(self2 - m);
      const float inv = 1.f / l;
      if (a.lse != nullptr && valid) a.lse[(size_t)slab * a.n + j] = n_kv > 0 ? m + log2f(l) : -INFINITY;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        if (n_kv > 0) {
          tmem_ld_x32_sync(tm_lane + kColO + c * 32, r);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = 0u;
        }
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          const uint32_t off = tile_chunk_offset(row, c * 4 + g);
          float vf[8];
          Elem<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4 *>(sK + off), vf);
          uint32_t o[4];
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            const float x0 = fmaf(w_self, vf[e], __uint_as_float(r[g * 8 + e])) * inv;
            const float x1 = fmaf(w_self, vf[e + 1], __uint_as_float(r[g * 8 + e + 1])) * inv;
            o[e >> 1] = pack_bf16x2(x0, x1);
          }
          *reinterpret_cast<uint4 *>(sV + off) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
      fence_proxy_async_smem();
    }
    named_barrier_sync(1, 128);
    if (ok && threadIdx.x == 64) {
      tma_store_3d(&tmO, sV, 0, j0, slab);           // rows past n are dropped by the tensor map
      tma_store_3d(&tmO, sV + kPfPanel, 64, j0, slab);
      tma_store_commit();
      tma_store_wait_read();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

bool prefill_tc_supported(const ag_layer_desc &d, const ag_cache &c) {
  return d.dtype == AG_BF16 && d.head_dim == 128 && c.pool_rows < ((int64_t)1 << 31) &&
         (int64_t)d.batch * d.heads * ((d.seq + kPfBM - 1) / kPfBM) < ((int64_t)1 << 31);
}

int launch_prefill_tc(const ag_layer_desc &d, const void *Q, const void *K, const void *V, const ag_cache &c,
                      const int32_t *prefix, float scale, void *O, float *lse, cudaStream_t st) {
  const int slabs = d.batch * d.heads;
  CUtensorMap tmQ, tmKd, tmVd, tmO, tmK, tmV;
  int rc;
  if ((rc = make_tmap_3d_bf16(&tmQ, Q, slabs, d.seq, kPfD, kPfBM, 64))) return rc;
  const int kv_slabs = d.batch * kv_heads_of(d);
  if ((rc = make_tmap_3d_bf16(&tmKd, K, kv_slabs, d.seq, kPfD, kPfBM, 64))) return rc;
  if ((rc = make_tmap_3d_bf16(&tmVd, V, kv_slabs, d.seq, kPfD, kPfBM, 64))) return rc;
  if ((rc = make_tmap_3d_bf16(&tmO, O, slabs, d.seq, kPfD, kPfBM, 64))) return rc;
  // an empty pool still needs a valid map: describe one row of the dense K / V instead (never read)
  const bool empty = c.pool_rows == 0;
  rc = make_tmap_2d_bf16(&tmK, empty ? K : c.k_rows, empty ? 1 : (uint64_t)c.pool_rows, kPfD, kPfD * 2, kPfBN, 64);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmV, empty ? V : c.v_rows, empty ? 1 : (uint64_t)c.pool_rows, kPfD, kPfD * 2, kPfBN, 64);
  if (rc) return rc;
  PrefillTcArgs a;
  a.prefix = prefix; a.row_off = c.row_off; a.len = c.len;
  a.n = d.seq; a.n_qtiles = (d.seq + kPfBM - 1) / kPfBM; a.slabs = slabs;
  a.heads = d.heads; a.kv_heads = kv_heads_of(d);
  a.scale_log2 = scale * 1.4426950408889634f;
  a.lse = lse;
  a.seq_lens = d.seq_lens;
  AG_CUDA_TRY(cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes));
  prefill_tc_kernel<<<a.n_qtiles * slabs, kPfThreads, kPfSmemBytes, st>>>(tmQ, tmKd, tmVd, tmO, tmK, tmV, a);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int prefill_tc_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
