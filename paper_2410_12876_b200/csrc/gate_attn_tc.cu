// MHA' of the Attention-Gate (Sec. 3.3) on the Blackwell tensor cores with
// float32-level accuracy.
//
// The gate's scores decide a hard threshold (Eq. 4), so bf16 rounding of Q', K',
// V' or of the attention weights would flip flags.  Every float32 operand x is
// therefore carried as a bf16 pair x = hi + lo (|x - hi - lo| <= 2^-17 |x|) and
// each product A B is evaluated as  Ahi Bhi + Ahi Blo + Alo Bhi  in the float32
// accumulator (the dropped lo*lo term is 2^-16 relative).
//
// Structure as in the prefill kernel: warp 0 TMA, warp 1 tcgen05.mma issue,
// warps 2..5 softmax with one row per thread.  A query tile is 128 queries of
// one (sequence, gate head); key tiles hold 64 keys (32 KB per K or V stage with
// the hi and lo halves), two stages each, so loads run a tile ahead of the MMAs.
//
// Work is the list of all (query tile, key tile) steps, query tiles in order
// and each one's key tiles in order.  The list is cut into equal segments, one
// CTA (one SM) each, so every SM gets the same number of steps whatever the
// shape of the causal triangle.  A segment crosses query tiles: the CTA handles
// its pieces one after the other, the loads of the next piece running under the
// tail of the current one.  Every piece leaves an un-normalised partial
// (O, m, l); gate_merge_out_kernel combines the pieces of a query tile and
// applies the gate's output layer and threshold.
//
// TMEM columns: S0 [0,64) S1 [128,192) O [256,384) Phi [384,448) Plo [448,512), each P half holding two
// tiles' weights (32 columns per tile).
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

constexpr int kGaThreads = 192;
constexpr int kGaBM = 128, kGaBN = 64, kGaD = 128;
constexpr int kGaPanel = 128 * 128;                  // Q: [128 rows][64 bf16]
constexpr int kGaTile = 2 * kGaPanel;                // 32 KB: Q hi or Q lo
constexpr int kGaKvPanel = kGaBN * 128;              // K / V: [64 rows][64 bf16] = 8 KB
constexpr int kGaKvTile = 2 * kGaKvPanel;            // 16 KB: one of hi / lo
constexpr int kGaKvStage = 2 * kGaKvTile;            // 32 KB: hi + lo
constexpr int kGaSmemBytes = 2 * kGaTile + 4 * kGaKvStage + 1024 + 256;   // Q + 2 K stages + 2 V stages
constexpr uint32_t kGaColS = 0, kGaColO = 256, kGaColPhi = 384, kGaColPlo = 448, kGaTmemCols = 512;
constexpr float kGaRescaleThreshold = 8.f;

constexpr int kGaMaxSeg = 256;       // segments at most (one per SM)
constexpr int kGaPieceCost = 3;      // set-up + epilogue of a piece, in half tile steps

struct GateAttnArgs {
  const int32_t *seq_lens;  // [B] or NULL: tokens past seq_lens[b] are padding
  float *part_o;            // [items, 128, 128] un-normalised partial outputs
  float *part_ml;           // [items, 128, 2]   running max (log2 units) and sum per row
  int n, n_qtiles, gate_heads, problems, GD, causal;
  int steps_per_prob;       // (query tile, key tile) steps of one (sequence, head)
  int total_steps;          // over all problems
  int n_seg;                // segments (= CTAs of the attention kernel)
  // Segment s covers steps [seg_begin[s], seg_begin[s + 1]) of the list.  Every boundary is even: a
  // piece starts on a 128-key boundary, so its first tile holds a key every row of the query tile
  // may see.  Segments are cut to equal cost, a piece counting as much as kGaPieceCost / 2 steps.
  int seg_begin[kGaMaxSeg + 1];
  float scale_log2;
};

// Key tiles query tile qt attends to, and the work items they are cut into.
// (key tiles hold 64 keys, query tiles 128 queries)
__host__ __device__ inline int ga_key_tiles(int qt, int n_qtiles, int causal) {
  return (kGaBM / kGaBN) * (causal ? qt + 1 : n_qtiles);
}
// First step of query tile qt within its problem's list.
__host__ __device__ inline int ga_first_step(int qt, int n_qtiles, int causal) {
  return causal ? qt * (qt + 1) : qt * 2 * n_qtiles;
}
// The piece of a segment that starts at global step x (x < x_end, the segment's end).
struct GaPiece {
  int prob, qt, kv_begin, n_kv;
};
__device__ inline GaPiece ga_piece(const GateAttnArgs &a, int x, int x_end) {
  GaPiece p;
  p.prob = x / a.steps_per_prob;
  const int y = x - p.prob * a.steps_per_prob;
  if (a.causal) {
    int qt = (int)((sqrtf(4.f * (float)y + 1.f) - 1.f) * 0.5f);
    while (qt > 0 && qt * (qt + 1) > y) --qt;
    while ((qt + 1) * (qt + 2) <= y) ++qt;
    p.qt = qt;
  } else {
    p.qt = y / (2 * a.n_qtiles);
  }
  p.kv_begin = y - ga_first_step(p.qt, a.n_qtiles, a.causal);
  const int tile_end = x - p.kv_begin + ga_key_tiles(p.qt, a.n_qtiles, a.causal);   // global end of the query tile
  p.n_kv = min(x_end, tile_end) - x;
  return p;
}
// A piece whose query tile lies wholly in its sequence's padding: nothing to compute (every role
// skips it the same way; the softmax role leaves an empty partial for the merge).
__device__ inline bool ga_padding_only(const GateAttnArgs &a, const GaPiece &p) {
  return a.seq_lens != nullptr && p.qt * kGaBM >= a.seq_lens[p.prob / a.gate_heads];
}
// Segment that holds global step x.
__device__ inline int ga_segment_of(const GateAttnArgs &a, int x) {
  int lo = 0, hi = a.n_seg - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (a.seg_begin[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}
// Partial slot of the piece of query tile (prob, qt) that lies in segment seg: consecutive pieces
// differ in the query tile, the segment or both, so the sum is unique and grows along the list.
__host__ __device__ inline int ga_slot(int prob, int qt, int n_qtiles, int seg) {
  return prob * n_qtiles + qt + seg;
}

__global__ void __launch_bounds__(kGaThreads, 1)
gate_attn_tc_kernel(const __grid_constant__ CUtensorMap tmHi, const __grid_constant__ CUtensorMap tmLo,
                    const __grid_constant__ CUtensorMap tmHiKv, const __grid_constant__ CUtensorMap tmLoKv,
                    const __grid_constant__ GateAttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;                    // [hi | lo]
  uint8_t *sK = sQ + 2 * kGaTile;        // [stage][hi | lo]
  uint8_t *sV = sK + 2 * kGaKvStage;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sV + 2 * kGaKvStage);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 3, *v_full = bars + 5, *v_empty = bars + 7;  // [2]
  uint64_t *s_full = bars + 9;           // [2]
  // p_ready[2], pv_done[2]: even / odd tiles.  P is double-buffered (32 of each half's 64 columns per tile), so
  // the weights of tile t are written while the P V of tile t - 1 runs; a softmax warp may be a tile ahead
  // of a slower one, never two (the scores of tile t + 2 exist only after every thread arrived for tile t).
  uint64_t *p_ready = bars + 11, *pv_done = bars + 13;
  uint64_t *q_empty = bars + 15, *o_free = bars + 16;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 17);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // This CTA's segment of the step list.  Every role walks its pieces with the same arithmetic;
  // tiles are numbered t = 0, 1, ... across the pieces (stage and S buffer t & 1, in their use
  // number t >> 1; P and the P V barrier in their use number t), pieces pc = 0, 1, ...
  const int x_begin = a.seg_begin[blockIdx.x];
  const int x_end = a.seg_begin[blockIdx.x + 1];

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
      mbar_init(&s_full[s], 1);
    }
    mbar_init(&p_ready[0], 128); mbar_init(&p_ready[1], 128);
    mbar_init(&pv_done[0], 1); mbar_init(&pv_done[1], 1);
    mbar_init(q_empty, 1);
    mbar_init(o_free, 128);
    fence_barrier_init();
    prefetch_tensormap(&tmHi); prefetch_tensormap(&tmLo);
    prefetch_tensormap(&tmHiKv); prefetch_tensormap(&tmLoKv);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kGaTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int t = 0;
      for (int x = x_begin, pc = 0; x < x_end && ok; ++pc) {      // pc counts the pieces that are computed
        const GaPiece pz = ga_piece(a, x, x_end);
        if (ga_padding_only(a, pz)) { x += pz.n_kv; --pc; continue; }
        const int b = pz.prob / a.gate_heads, g = pz.prob % a.gate_heads, j0 = pz.qt * kGaBM;
        const int xq = g * kGaD, xk = a.GD + g * kGaD, xv = 2 * a.GD + g * kGaD;   // columns in [Q' | K' | V']
        ok = mbar_wait(q_empty, (pc & 1) ^ 1);       // the previous piece's last Q K^T has read Q
        if (!ok) break;
        mbar_arrive_expect_tx(q_full, 2 * kGaTile);
        tma_load_3d(sQ, &tmHi, q_full, xq, j0, b);
        tma_load_3d(sQ + kGaPanel, &tmHi, q_full, xq + 64, j0, b);
        tma_load_3d(sQ + kGaTile, &tmLo, q_full, xq, j0, b);
        tma_load_3d(sQ + kGaTile + kGaPanel, &tmLo, q_full, xq + 64, j0, b);
        auto load_kv = [&](uint8_t *dst, uint64_t *bar, int xc, int y) {
          mbar_arrive_expect_tx(bar, kGaKvStage);
          tma_load_3d(dst, &tmHiKv, bar, xc, y, b);
          tma_load_3d(dst + kGaKvPanel, &tmHiKv, bar, xc + 64, y, b);
          tma_load_3d(dst + kGaKvTile, &tmLoKv, bar, xc, y, b);
          tma_load_3d(dst + kGaKvTile + kGaKvPanel, &tmLoKv, bar, xc + 64, y, b);
        };
        for (int i = 0; i < pz.n_kv; ++i, ++t) {
          const int st = t & 1;
          const uint32_t ph = (t >> 1) & 1;
          const int y = (pz.kv_begin + i) * kGaBN;
          if (!mbar_wait(&k_empty[st], ph ^ 1)) { ok = false; break; }
          load_kv(sK + st * kGaKvStage, &k_full[st], xk, y);
          if (!mbar_wait(&v_empty[st], ph ^ 1)) { ok = false; break; }
          load_kv(sV + st * kGaKvStage, &v_full[st], xv, y);
        }
        x += pz.n_kv;
      }
    }
  } else if (warp == 1) {
    // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
    constexpr uint32_t idesc_qk = idesc_bf16_f32(kGaBM, kGaBN, false, false);
    constexpr uint32_t idesc_pv = idesc_bf16_f32(kGaBM, kGaD, false, true);
    const uint64_t dq = desc_kmajor_sw128(smem_u32(sQ)), dk = desc_kmajor_sw128(smem_u32(sK));
    const uint64_t dv = desc_mnmajor_sw128(smem_u32(sV), kGaKvPanel);
    const uint32_t q_lo = (uint32_t)dq, q_hi = (uint32_t)(dq >> 32);
    const uint32_t k_lo = (uint32_t)dk, k_hi = (uint32_t)(dk >> 32);
    const uint32_t v_lo = (uint32_t)dv, v_hi = (uint32_t)(dv >> 32);
    auto issue_qk = [&](int t, bool last) -> bool {   // t: tile number across the pieces
      const int st = t & 1;
      if (!mbar_wait(&k_full[st], (t >> 1) & 1)) return false;
      tc_fence_after_sync();
      const uint32_t d = tmem + kGaColS + st * 128;
      const uint32_t kb = k_lo + ((st * kGaKvStage) >> 4);
      if (elect_one()) {
        // Qhi Khi + Qhi Klo + Qlo Khi
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const uint32_t qa = q_lo + ((t == 2 ? kGaTile : 0) >> 4), ka = kb + ((t == 1 ? kGaKvTile : 0) >> 4);
#pragma unroll
          for (int k = 0; k < kGaD / 16; ++k)
            mma_ss_lohi(d, qa + (((k >> 2) * kGaPanel + (k & 3) * 32) >> 4), q_hi,
                        ka + (((k >> 2) * kGaKvPanel + (k & 3) * 32) >> 4), k_hi, idesc_qk, (t | k) != 0);
        }
        mma_commit(&k_empty[st]);
        mma_commit(&s_full[st]);
        if (last) mma_commit(q_empty);               // Q may be replaced by the next piece's
      }
      __syncwarp();
      return true;
    };
    bool ok = true;
    int t0 = 0;                                      // tile number of the piece's first tile
    for (int x = x_begin, pc = 0; x < x_end && ok; ++pc) {        // pc counts the pieces that are computed
      const GaPiece pz = ga_piece(a, x, x_end);
      const int n_kv = pz.n_kv;
      if (ga_padding_only(a, pz)) { x += n_kv; --pc; continue; }
      ok = mbar_wait(q_full, pc & 1);
      ok = ok && issue_qk(t0, n_kv == 1);
      for (int i = 0; i < n_kv && ok; ++i) {
      const int t = t0 + i;
      if (i + 1 < n_kv) ok = issue_qk(t + 1, i + 2 == n_kv);
      if (!ok) break;
      const int st = t & 1;
      if (!mbar_wait(&p_ready[t & 1], (t >> 1) & 1)) { ok = false; break; }
      if (!mbar_wait(&v_full[st], (t >> 1) & 1)) { ok = false; break; }
      // the first P V of a piece overwrites O: the previous piece's epilogue must have read it
      if (i == 0 && pc > 0 && !mbar_wait(o_free, (pc - 1) & 1)) { ok = false; break; }
      tc_fence_after_sync();
      const uint32_t vb = v_lo + ((st * kGaKvStage) >> 4);
      if (elect_one()) {
        // Phi Vhi + Phi Vlo + Plo Vhi
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const uint32_t pa = tmem + (t == 2 ? kGaColPlo : kGaColPhi) + st * (kGaBN / 2), va = vb + ((t == 1 ? kGaKvTile : 0) >> 4);
#pragma unroll
          for (int k = 0; k < kGaBN / 16; ++k)
            mma_ts_lohi(tmem + kGaColO, pa + k * 8, va + ((k * 2048) >> 4), v_hi, idesc_pv, (i | t | k) != 0);
        }
        mma_commit(&v_empty[st]);
        mma_commit(&pv_done[st]);
      }
      __syncwarp();
      }
      t0 += n_kv;
      x += n_kv;
    }
  } else {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    bool ok = true;
    int t0 = 0;                                      // tile number of the piece's first tile

    for (int x = x_begin; x < x_end && ok;) {
    const GaPiece pz = ga_piece(a, x, x_end);
    const int n_kv = pz.n_kv, kv_begin = pz.kv_begin;
    const int j = pz.qt * kGaBM + row;
    const bool valid = j < a.n;
    const int jc = min(j, a.n - 1);
    // keys below bound are visible (bidirectional: the sequence's own tokens, not its padding)
    const int seq_len = a.seq_lens ? a.seq_lens[pz.prob / a.gate_heads] : a.n;
    const int bound = a.causal ? jc + 1 : seq_len;
    float m = -INFINITY, l = 0.f;
    if (ga_padding_only(a, pz)) {
      // padding only: an empty partial (weight 0 in the merge; the merge gives padding flag 0 anyway)
      const size_t it = (size_t)ga_slot(pz.prob, pz.qt, a.n_qtiles, (int)blockIdx.x);
      if (valid) {
        float *op = a.part_o + (it * kGaBM + row) * kGaD;
#pragma unroll 4
        for (int e = 0; e < kGaD; e += 4) *reinterpret_cast<uint4 *>(op + e) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<float2 *>(a.part_ml + (it * kGaBM + row) * 2) = make_float2(m, l);
      }
      x += n_kv;
      continue;
    }

    for (int i = 0; i < n_kv && ok; ++i) {
      const int t = t0 + i;
      ok = mbar_wait(&s_full[t & 1], (t >> 1) & 1);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tS = tm_lane + kGaColS + (t & 1) * 128;
      const int nvalid = min(max(bound - (kv_begin + i) * kGaBN, 0), kGaBN);
      const bool full = nvalid >= kGaBN;

      uint32_t r[kGaBN];
      tmem_ld_x64_sync(tS, r);
      if (!full) {
#pragma unroll
        for (int e = 0; e < kGaBN; ++e)
          if (e >= nvalid) r[e] = 0xff800000u;        // -inf: weight 0 below
      }
      float mx[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) mx[q] = __uint_as_float(r[q]);
#pragma unroll
      for (int e = 8; e < kGaBN; e += 8)
#pragma unroll
        for (int q = 0; q < 8; ++q) mx[q] = fmaxf(mx[q], __uint_as_float(r[e + q]));
      float tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                         fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
      tmax *= a.scale_log2;
      // The first tile of a piece holds a key visible to every row (key 0, or a tile wholly before
      // the query tile) - unless the sequence is shorter than its padded length and the bidirectional
      // MHA' has no key in this piece at all: m then stays -inf, every weight is 0, and the piece's
      // partial (m = -inf, l = 0, O = 0) drops out of the merge.
      float m_new;
      if (i == 0) m_new = tmax;
      else m_new = (tmax > m + kGaRescaleThreshold) ? tmax : m;
      const bool rescale = (i > 0) && __any_sync(0xffffffffu, m_new != m);
      const float alpha = (i == 0 || m == -INFINITY) ? 0.f : fast_exp2(m - m_new);
      l *= alpha;
      const float m_exp = m_new == -INFINITY ? 0.f : m_new;    // exponent offset: keeps -inf - (-inf) out

      // Only a rescale of O has to wait for the P V of tile t - 1 (the next phase of that barrier is the P V of
      // tile t + 1, which cannot have been issued yet: the parity is unambiguous)
      if (rescale) {
        ok = mbar_wait(&pv_done[(t - 1) & 1], ((t - 1) >> 1) & 1);
        if (!ok) break;
        tc_fence_after_sync();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t r[32];
          tmem_ld_x32_sync(tm_lane + kGaColO + c * 32, r);
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
          tmem_st_x32(tm_lane + kGaColO + c * 32, r);
        }
      }
      // this tile's P buffer was last read by the P V of tile t - 2
      if (t >= 2) {
        ok = mbar_wait(&pv_done[t & 1], ((t >> 1) & 1) ^ 1);
        if (!ok) break;
        tc_fence_after_sync();
      }

      float rs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < kGaBN / 16; ++c) {
        uint32_t ph[8], pl[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e]), a.scale_log2, -m_exp));
          const float p1 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e + 1]), a.scale_log2, -m_exp));
          rs[(e >> 1) & 3] += p0 + p1;
          float h0, l0, h1, l1;
          split_bf16(p0, h0, l0);
          split_bf16(p1, h1, l1);
          ph[e >> 1] = pack_bf16x2(h0, h1);
          pl[e >> 1] = pack_bf16x2(l0, l1);
        }
        tmem_st_x8(tm_lane + kGaColPhi + (t & 1) * (kGaBN / 2) + c * 8, ph);
        tmem_st_x8(tm_lane + kGaColPlo + (t & 1) * (kGaBN / 2) + c * 8, pl);
      }
      const float rowsum = (rs[0] + rs[1]) + (rs[2] + rs[3]);
      l += rowsum;
      m = m_new;
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(&p_ready[t & 1]);
    }

    if (ok) {
      ok = mbar_wait(&pv_done[(t0 + n_kv - 1) & 1], ((t0 + n_kv - 1) >> 1) & 1);
      tc_fence_after_sync();
    }
    if (ok) {
      const size_t it = (size_t)ga_slot(pz.prob, pz.qt, a.n_qtiles, (int)blockIdx.x);
      float *op = a.part_o + (it * kGaBM + row) * kGaD;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld_x32_sync(tm_lane + kGaColO + c * 32, r);
        if (c == 3) {                                // O is in registers: the next piece may overwrite it
          tc_fence_before_sync();
          mbar_arrive(o_free);
        }
        if (valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<uint4 *>(op + c * 32 + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
        }
      }
      if (valid) *reinterpret_cast<float2 *>(a.part_ml + (it * kGaBM + row) * 2) = make_float2(m, l);
    }
    t0 += n_kv;
    x += n_kv;
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, kGaTmemCols);
}

bool gate_attn_tc_supported(const ag_layer_desc &d) {
  const int GD = d.gate_heads * d.gate_head_dim;
  return d.dtype == AG_BF16 && d.gate_head_dim == 128 && gate_proj_tc_supported(d.hidden, GD);
}

// The split-K merge of MHA' and the gate's output layer in one pass (Eq. 3, Eq. 4):
//   H'[t, g * 128 + c] = sum_s w_s O_s[r, c] / sum_s w_s l_s,  w_s = 2^(m_s - max_s m_s)
//   s[t, i] = H'[t, :] Wo_g[:, i];  flag = s + gamma_i > logit(tau)
// One CTA = 16 tokens, one warp per token.  A warp merges the token's row of every gate head
// (a lane per four columns: every access is one 512-byte row) into shared memory; then warp w
// takes four tokens and a quarter of the reduction, a lane per head, in rounds of 32 heads,
// against a [GD][32] slice of Wo staged in shared memory.  H' never goes to global memory.
constexpr int kMoTokens = 16, kMoThreads = kMoTokens * 32;
template <typename T>
__global__ void __launch_bounds__(kMoThreads)
gate_merge_out_kernel(const __grid_constant__ GateAttnArgs a, const T *__restrict__ Wo, const float *__restrict__ gamma,
                      float logit_tau, int h, float *__restrict__ scores, uint8_t *__restrict__ flags) {
  extern __shared__ __align__(16) unsigned char mo_smem[];
  float *Hs = reinterpret_cast<float *>(mo_smem);                                   // [16][GD]
  T *Ws = reinterpret_cast<T *>(mo_smem + sizeof(float) * kMoTokens * a.GD);       // [GD][32]
  float *red = reinterpret_cast<float *>(mo_smem + sizeof(float) * kMoTokens * a.GD + sizeof(T) * a.GD * 32);  // [4][16][32]
  const int tiles_per_seq = (a.n + kMoTokens - 1) / kMoTokens;
  const int b = blockIdx.x / tiles_per_seq, t0 = (blockIdx.x % tiles_per_seq) * kMoTokens;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = t0 + warp;
  float *hrow = Hs + warp * a.GD;
  // The CTA's 16 tokens lie in one query tile: which segments hold its pieces is looked up once per
  // gate head (a binary search over the boundaries in constant memory), by one thread each.
  int *seg_first = reinterpret_cast<int *>(red);     // [gate_heads] first segment, then [gate_heads] piece count
  {
    const int qt = t0 / kGaBM;
    const int y0 = ga_first_step(qt, a.n_qtiles, a.causal), y1 = y0 + ga_key_tiles(qt, a.n_qtiles, a.causal);
    for (int g = threadIdx.x; g < a.gate_heads; g += kMoThreads) {
      const int prob = b * a.gate_heads + g;
      // the query tile's steps [x0, x1) of the list lie in segments seg0 .. seg1, one piece in each
      const int x0 = prob * a.steps_per_prob + y0, x1 = prob * a.steps_per_prob + y1;
      const int seg0 = ga_segment_of(a, x0);
      seg_first[g] = seg0;
      seg_first[a.gate_heads + g] = ga_segment_of(a, x1 - 1) - seg0 + 1;
    }
  }
  __syncthreads();
  if (t < a.n) {
    const int qt = t / kGaBM, r = t % kGaBM;
    // four gate heads at a time, so that their loads are in flight together
    for (int g0 = 0; g0 < a.gate_heads; g0 += 4) {
      size_t row0[4];
      int ns[4];
      float mmax[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int g = min(g0 + u, a.gate_heads - 1), prob = b * a.gate_heads + g;
        ns[u] = seg_first[a.gate_heads + g];
        row0[u] = (size_t)ga_slot(prob, qt, a.n_qtiles, seg_first[g]) * kGaBM + r;   // + s * 128 per piece
        mmax[u] = -INFINITY;
        for (int s = lane; s < ns[u]; s += 32) mmax[u] = fmaxf(mmax[u], a.part_ml[(row0[u] + (size_t)s * kGaBM) * 2]);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mmax[u] = fmaxf(mmax[u], __shfl_xor_sync(0xffffffffu, mmax[u], off));
      float4 acc[4];
      float lsum[4];
      int ns_max = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) { acc[u] = make_float4(0.f, 0.f, 0.f, 0.f); lsum[u] = 0.f; ns_max = max(ns_max, ns[u]); }
      for (int s = 0; s < ns_max; ++s) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (s < ns[u]) {
            const float2 ml = *reinterpret_cast<const float2 *>(a.part_ml + (row0[u] + (size_t)s * kGaBM) * 2);
            const float4 o = *reinterpret_cast<const float4 *>(a.part_o + (row0[u] + (size_t)s * kGaBM) * kGaD + lane * 4);
            const float w = fast_exp2(ml.x - mmax[u]);
            acc[u].x = fmaf(w, o.x, acc[u].x); acc[u].y = fmaf(w, o.y, acc[u].y);
            acc[u].z = fmaf(w, o.z, acc[u].z); acc[u].w = fmaf(w, o.w, acc[u].w);
            lsum[u] = fmaf(w, ml.y, lsum[u]);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (g0 + u < a.gate_heads) {
          const float inv = 1.f / lsum[u];
          *reinterpret_cast<float4 *>(hrow + (g0 + u) * kGaD + lane * 4) =
              make_float4(acc[u].x * inv, acc[u].y * inv, acc[u].z * inv, acc[u].w * inv);
        }
      }
    }
  }
  for (int i0 = 0; i0 < h; i0 += 32) {
    __syncthreads();                                 // H' rows complete; previous slice of Wo consumed
    if (sizeof(T) == 2 && (h & 7) == 0) {            // 16-byte pieces of the rows of Wo
      for (int x = threadIdx.x; x < a.GD * 4; x += kMoThreads) {
        const int c = x >> 2, i = i0 + (x & 3) * 8;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i < h) v = ldg128(Wo + (size_t)c * h + i);
        *reinterpret_cast<uint4 *>(Ws + c * 32 + (x & 3) * 8) = v;
      }
    } else {
      for (int x = threadIdx.x; x < a.GD * 32; x += kMoThreads) {
        const int c = x >> 5, i = i0 + (x & 31);
        Ws[x] = i < h ? Wo[(size_t)c * h + i] : T(0.f);
      }
    }
    __syncthreads();
    {
      // warp w: tokens 4 (w & 3) .. + 3 against head `lane` over a quarter of the reduction,
      // c in [cq, cq + 1) GD / 4; per four steps four broadcast float4 of H' and four values of Wo
      // feed sixteen FMAs.  The quarters are added in a fixed order below.
      const int tq = warp & 3, cq = warp >> 2;
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      const float *h4 = Hs + tq * 4 * a.GD;
      const int c_begin = cq * (a.GD / 4), c_end = c_begin + a.GD / 4;    // GD is a multiple of 128
#pragma unroll 4
      for (int c = c_begin; c < c_end; c += 4) {
        float w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) w[k] = Elem<T>::load(Ws + (c + k) * 32 + lane);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 x = *reinterpret_cast<const float4 *>(h4 + q * a.GD + c);
          acc[q] = fmaf(x.x, w[0], acc[q]);
          acc[q] = fmaf(x.y, w[1], acc[q]);
          acc[q] = fmaf(x.z, w[2], acc[q]);
          acc[q] = fmaf(x.w, w[3], acc[q]);
        }
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) red[(cq * kMoTokens + tq * 4 + q) * 32 + lane] = acc[q];
    }
    __syncthreads();
    {
      // thread (token = warp, head = lane): the four quarters in order
      const float *rp = red + warp * 32 + lane;
      const float sc = ((rp[0] + rp[kMoTokens * 32]) + rp[2 * kMoTokens * 32]) + rp[3 * kMoTokens * 32];
      const int i = i0 + lane;
      if (i < h && t < a.n) {
        const size_t o = ((size_t)b * h + i) * a.n + t;
        const bool padding = a.seq_lens && t >= a.seq_lens[b];
        if (scores) scores[o] = sc;
        flags[o] = !padding && (sc + (gamma ? gamma[i] : 0.f)) > logit_tau ? 1 : 0;
      }
    }
  }
}

// Cuts the step list into at most `n_target` segments of about equal cost (2 per tile step,
// kGaPieceCost per piece) and writes their boundaries; returns the number of segments.
static int cut_segments(int problems, int nq, int causal, int n_target, int target, int *seg_begin) {
  int n = 0, cur = 0, x = 0;
  seg_begin[n++] = 0;
  for (int prob = 0; prob < problems; ++prob)
    for (int qt = 0; qt < nq; ++qt) {
      int r = ga_key_tiles(qt, nq, causal);
      while (r > 0) {
        if (cur > 0 && cur + kGaPieceCost + 4 > target) {      // not even a two-tile piece fits: new segment
          if (n >= n_target) return n_target + 1;
          seg_begin[n++] = x;
          cur = 0;
        }
        cur += kGaPieceCost;
        int fit = ((target - cur) / 2) & ~1;
        if (fit < 2) fit = 2;
        const int take = r < fit ? r : fit;
        cur += 2 * take; x += take; r -= take;
        if (r > 0) {                                           // segment full inside the query tile
          if (n >= n_target) return n_target + 1;
          seg_begin[n++] = x;
          cur = 0;
        }
      }
    }
  seg_begin[n] = x;
  return n;                                                    // seg_begin[0 .. n]
}

struct GateAttnPlan {
  int steps_per_prob, total_steps, n_seg;
  int seg_begin[kGaMaxSeg + 1];
};
static int gate_attn_plan(const ag_layer_desc &d, GateAttnPlan &p) {
  static int sm_count[64] = {0};                     // per device, read once
  int dev = 0;
  AG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return AG_ERR_UNSUPPORTED;
  if (sm_count[dev] == 0) {
    int v = 0;
    AG_CUDA_TRY(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
    sm_count[dev] = v < 1 ? 1 : (v > kGaMaxSeg ? kGaMaxSeg : v);
  }
  const int nq = (d.seq + kGaBM - 1) / kGaBM, problems = d.batch * d.gate_heads;
  const long long per = d.gate_causal ? (long long)nq * (nq + 1) : 2LL * nq * nq;
  const long long total = per * problems;
  if (total >= (1LL << 28)) return AG_ERR_UNSUPPORTED;
  p.steps_per_prob = (int)per;
  p.total_steps = (int)total;
  const int n_target = sm_count[dev];
  // cost per segment: raised until the cuts fit into n_target segments
  long long target = (2 * total + (long long)kGaPieceCost * ((long long)problems * nq + n_target) + n_target - 1) / n_target;
  if (target < kGaPieceCost + 4) target = kGaPieceCost + 4;
  for (;;) {
    p.n_seg = cut_segments(problems, nq, d.gate_causal, n_target, (int)target, p.seg_begin);
    if (p.n_seg <= n_target) break;
    target += 1 + target / 64;
  }
  return AG_OK;
}

size_t gate_attn_partial_bytes(const ag_layer_desc &d) {
  // one slot per piece: query tiles + segments, whatever the device (no device is asked here)
  const size_t nq = (d.seq + kGaBM - 1) / kGaBM;
  const size_t slots = (size_t)d.batch * d.gate_heads * nq + kGaMaxSeg;
  return align_up(slots * kGaBM * kGaD * sizeof(float), 256) + align_up(slots * kGaBM * 2 * sizeof(float), 256);
}

int launch_gate_attn_tc(const ag_layer_desc &d, const void *qkv_hi, const void *qkv_lo, void *partials,
                        const void *Wo, const float *gamma, float logit_tau, float *scores, uint8_t *flags,
                        cudaStream_t st) {
  const int GD = d.gate_heads * d.gate_head_dim;
  CUtensorMap tmHi, tmLo;
  int rc = make_tmap_3d_bf16(&tmHi, qkv_hi, d.batch, d.seq, 3 * GD, kGaBM, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmLo, qkv_lo, d.batch, d.seq, 3 * GD, kGaBM, 64);
  if (rc) return rc;
  CUtensorMap tmHiKv, tmLoKv;
  if ((rc = make_tmap_3d_bf16(&tmHiKv, qkv_hi, d.batch, d.seq, 3 * GD, kGaBN, 64))) return rc;
  if ((rc = make_tmap_3d_bf16(&tmLoKv, qkv_lo, d.batch, d.seq, 3 * GD, kGaBN, 64))) return rc;
  GateAttnArgs a;
  a.seq_lens = d.seq_lens;
  a.n = d.seq; a.n_qtiles = (d.seq + kGaBM - 1) / kGaBM;
  a.gate_heads = d.gate_heads; a.problems = d.batch * d.gate_heads; a.GD = GD; a.causal = d.gate_causal;
  static thread_local GateAttnPlan plan;             // 1 KB of boundaries: not on the stack of every call
  if ((rc = gate_attn_plan(d, plan))) return rc;
  a.steps_per_prob = plan.steps_per_prob; a.total_steps = plan.total_steps; a.n_seg = plan.n_seg;
  for (int i = 0; i <= plan.n_seg; ++i) a.seg_begin[i] = plan.seg_begin[i];
  const size_t slots = (size_t)a.problems * a.n_qtiles + kGaMaxSeg;
  a.part_o = static_cast<float *>(partials);
  a.part_ml = reinterpret_cast<float *>(static_cast<char *>(partials) +
                                        align_up(slots * kGaBM * kGaD * sizeof(float), 256));
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kGaD));
  AG_CUDA_TRY(cudaFuncSetAttribute(gate_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGaSmemBytes));
  gate_attn_tc_kernel<<<(unsigned)plan.n_seg, kGaThreads, kGaSmemBytes, st>>>(tmHi, tmLo, tmHiKv, tmLoKv, a);
  AG_LAUNCH_CHECK();
  const size_t mo_smem = sizeof(float) * kMoTokens * GD + sizeof(__nv_bfloat16) * GD * 32 + sizeof(float) * 4 * kMoTokens * 32;
  auto mo = gate_merge_out_kernel<__nv_bfloat16>;
  AG_CUDA_TRY(cudaFuncSetAttribute(mo, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mo_smem));
  const int blocks = d.batch * ((d.seq + kMoTokens - 1) / kMoTokens);
  mo<<<blocks, kMoThreads, mo_smem, st>>>(a, static_cast<const __nv_bfloat16 *>(Wo), gamma, logit_tau, kv_heads_of(d),
                                          scores, flags);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int gate_attn_tc_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
