// MHA' of the Attention-Gate (Sec. 3.3) on the Blackwell tensor cores with
// float32-level accuracy.
//
// The gate's scores decide a hard threshold (Eq. 4), so bf16 rounding of Q', K',
// V' or of the attention weights would flip flags.  Every float32 operand x is
// therefore carried as a bf16 pair x = hi + lo (|x - hi - lo| <= 2^-17 |x|) and
// each product A B is evaluated as  Ahi Bhi + Ahi Blo + Alo Bhi  in the float32
// accumulator (the dropped lo*lo term is 2^-16 relative).
//
// One CTA = 128 queries of one (sequence, gate head).  Structure as in the
// prefill kernel: warp 0 TMA, warp 1 tcgen05.mma issue, warps 2..5 softmax with
// one row per thread.  K and V tiles are single-buffered: the K load of tile
// i + 2 overlaps P V of tile i and the V load of tile i + 1 overlaps Q K^T of
// tile i + 2.
//
// TMEM columns: S0 [0,128) S1 [128,256) O [256,384) Phi [384,448) Plo [448,512).
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

constexpr int kGaThreads = 192;
constexpr int kGaBM = 128, kGaBN = 128, kGaD = 128;
constexpr int kGaPanel = 128 * 128;                  // [128 rows][64 bf16]
constexpr int kGaTile = 2 * kGaPanel;                // 32 KB: one of hi / lo
constexpr int kGaSmemBytes = 6 * kGaTile + 1024 + 256;
constexpr uint32_t kGaColS = 0, kGaColO = 256, kGaColPhi = 384, kGaColPlo = 448, kGaTmemCols = 512;
constexpr float kGaRescaleThreshold = 8.f;

struct GateAttnArgs {
  float *H;                 // [B * n, GD]
  int n, n_qtiles, gate_heads, problems, GD, causal;
  float scale_log2;
};

__global__ void __launch_bounds__(kGaThreads, 1)
gate_attn_tc_kernel(const __grid_constant__ CUtensorMap tmHi, const __grid_constant__ CUtensorMap tmLo,
                    const GateAttnArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;                    // [hi | lo]
  uint8_t *sK = sQ + 2 * kGaTile;
  uint8_t *sV = sK + 2 * kGaTile;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sV + 2 * kGaTile);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 2, *v_full = bars + 3, *v_empty = bars + 4;
  uint64_t *s_full = bars + 5;           // [2]
  uint64_t *p_ready = bars + 7, *pv_done = bars + 8;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 9);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int qt = a.n_qtiles - 1 - (int)(blockIdx.x / a.problems);
  const int prob = blockIdx.x % a.problems;
  const int b = prob / a.gate_heads, g = prob % a.gate_heads;
  const int j0 = qt * kGaBM;
  const int n_kv = a.causal ? qt + 1 : a.n_qtiles;
  const int xq = g * kGaD, xk = a.GD + g * kGaD, xv = 2 * a.GD + g * kGaD;   // columns in [Q' | K' | V']

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(k_full, 1); mbar_init(k_empty, 1);
    mbar_init(v_full, 1); mbar_init(v_empty, 1);
    mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1);
    mbar_init(p_ready, 128);
    mbar_init(pv_done, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmHi); prefetch_tensormap(&tmLo);
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
      auto load_tile = [&](uint8_t *dst, uint64_t *bar, int x, int y) {
        mbar_arrive_expect_tx(bar, 2 * kGaTile);
        tma_load_3d(dst, &tmHi, bar, x, y, b);
        tma_load_3d(dst + kGaPanel, &tmHi, bar, x + 64, y, b);
        tma_load_3d(dst + kGaTile, &tmLo, bar, x, y, b);
        tma_load_3d(dst + kGaTile + kGaPanel, &tmLo, bar, x + 64, y, b);
      };
      load_tile(sQ, q_full, xq, j0);
      for (int i = 0; i < n_kv; ++i) {
        const uint32_t ph = i & 1;
        if (!mbar_wait(k_empty, ph ^ 1)) break;
        load_tile(sK, k_full, xk, i * kGaBN);
        if (!mbar_wait(v_empty, ph ^ 1)) break;
        load_tile(sV, v_full, xv, i * kGaBN);
      }
    }
  } else if (warp == 1) {
    // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
    constexpr uint32_t idesc_qk = idesc_bf16_f32(kGaBM, kGaBN, false, false);
    constexpr uint32_t idesc_pv = idesc_bf16_f32(kGaBM, kGaD, false, true);
    const uint64_t dq = desc_kmajor_sw128(smem_u32(sQ)), dk = desc_kmajor_sw128(smem_u32(sK));
    const uint64_t dv = desc_mnmajor_sw128(smem_u32(sV), kGaPanel);
    const uint32_t q_lo = (uint32_t)dq, q_hi = (uint32_t)(dq >> 32);
    const uint32_t k_lo = (uint32_t)dk, k_hi = (uint32_t)(dk >> 32);
    const uint32_t v_lo = (uint32_t)dv, v_hi = (uint32_t)(dv >> 32);
    auto issue_qk = [&](int i) -> bool {
      if (!mbar_wait(k_full, i & 1)) return false;
      tc_fence_after_sync();
      const uint32_t d = tmem + kGaColS + (i & 1) * 128;
      if (elect_one()) {
        // Qhi Khi + Qhi Klo + Qlo Khi
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const uint32_t qa = q_lo + ((t == 2 ? kGaTile : 0) >> 4), ka = k_lo + ((t == 1 ? kGaTile : 0) >> 4);
#pragma unroll
          for (int k = 0; k < kGaD / 16; ++k) {
            const uint32_t off = ((k >> 2) * kGaPanel + (k & 3) * 32) >> 4;
            mma_ss_lohi(d, qa + off, q_hi, ka + off, k_hi, idesc_qk, (t | k) != 0);
          }
        }
        mma_commit(k_empty);
        mma_commit(&s_full[i & 1]);
      }
      __syncwarp();
      return true;
    };
    bool ok = mbar_wait(q_full, 0);
    ok = ok && issue_qk(0);
    for (int i = 0; i < n_kv && ok; ++i) {
      if (i + 1 < n_kv) ok = issue_qk(i + 1);
      if (!ok) break;
      if (!mbar_wait(p_ready, i & 1)) { ok = false; break; }
      if (!mbar_wait(v_full, i & 1)) { ok = false; break; }
      tc_fence_after_sync();
      if (elect_one()) {
        // Phi Vhi + Phi Vlo + Plo Vhi
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const uint32_t pa = tmem + (t == 2 ? kGaColPlo : kGaColPhi), va = v_lo + ((t == 1 ? kGaTile : 0) >> 4);
#pragma unroll
          for (int k = 0; k < kGaBN / 16; ++k)
            mma_ts_lohi(tmem + kGaColO, pa + k * 8, va + ((k * 2048) >> 4), v_hi, idesc_pv, (i | t | k) != 0);
        }
        mma_commit(v_empty);
        mma_commit(pv_done);
      }
      __syncwarp();
    }
  } else {
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const int j = j0 + row;
    const bool valid = j < a.n;
    const int jc = min(j, a.n - 1);
    const int bound = a.causal ? jc + 1 : a.n;       // keys t < bound are visible
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    float m = -INFINITY, l = 0.f;
    bool ok = true;

    for (int i = 0; i < n_kv && ok; ++i) {
      ok = mbar_wait(&s_full[i & 1], (i >> 1) & 1);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t tS = tm_lane + kGaColS + (i & 1) * 128;
      const int nvalid = min(max(bound - i * kGaBN, 0), kGaBN);
      const bool full = nvalid >= kGaBN;

      uint32_t r[128];
      tmem_ld_x128_sync(tS, r);
      if (!full) {
#pragma unroll
        for (int e = 0; e < 128; ++e)
          if (e >= nvalid) r[e] = 0xff800000u;        // -inf: weight 0 below
      }
      float mx[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) mx[q] = __uint_as_float(r[q]);
#pragma unroll
      for (int e = 8; e < 128; e += 8)
#pragma unroll
        for (int q = 0; q < 8; ++q) mx[q] = fmaxf(mx[q], __uint_as_float(r[e + q]));
      float tmax = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                         fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
      tmax *= a.scale_log2;
      // tile 0 always holds key 0, visible to every row, so m is finite from here on
      float m_new;
      if (i == 0) m_new = tmax;
      else m_new = (tmax > m + kGaRescaleThreshold) ? tmax : m;
      const bool rescale = (i > 0) && __any_sync(0xffffffffu, m_new != m);
      const float alpha = (i == 0) ? 0.f : fast_exp2(m - m_new);
      l *= alpha;

      if (i > 0) {
        ok = mbar_wait(pv_done, (i - 1) & 1);
        if (!ok) break;
        tc_fence_after_sync();
        if (rescale) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            tmem_ld_x32_sync(tm_lane + kGaColO + c * 32, r);
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
            tmem_st_x32(tm_lane + kGaColO + c * 32, r);
          }
        }
      }

      float rs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t ph[8], pl[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e]), a.scale_log2, -m_new));
          const float p1 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e + 1]), a.scale_log2, -m_new));
          rs[(e >> 1) & 3] += p0 + p1;
          float h0, l0, h1, l1;
          split_bf16(p0, h0, l0);
          split_bf16(p1, h1, l1);
          ph[e >> 1] = pack_bf16x2(h0, h1);
          pl[e >> 1] = pack_bf16x2(l0, l1);
        }
        tmem_st_x8(tm_lane + kGaColPhi + c * 8, ph);
        tmem_st_x8(tm_lane + kGaColPlo + c * 8, pl);
      }
      const float rowsum = (rs[0] + rs[1]) + (rs[2] + rs[3]);
      l += rowsum;
      m = m_new;
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(p_ready);
    }

    if (ok) {
      ok = mbar_wait(pv_done, (n_kv - 1) & 1);
      tc_fence_after_sync();
    }
    if (ok) {
      const float inv = 1.f / l;
      float *hp = a.H + ((size_t)b * a.n + jc) * a.GD + g * kGaD;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld_x32_sync(tm_lane + kGaColO + c * 32, r);
        if (valid) {
#pragma unroll
          for (int e = 0; e < 32; e += 4)
            *reinterpret_cast<float4 *>(hp + c * 32 + e) =
                make_float4(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv,
                            __uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
        }
      }
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

int launch_gate_attn_tc(const ag_layer_desc &d, const void *qkv_hi, const void *qkv_lo, float *hcat,
                        cudaStream_t st) {
  const int GD = d.gate_heads * d.gate_head_dim;
  CUtensorMap tmHi, tmLo;
  int rc = make_tmap_3d_bf16(&tmHi, qkv_hi, d.batch, d.seq, 3 * GD, kGaBM, 64);
  if (rc) return rc;
  rc = make_tmap_3d_bf16(&tmLo, qkv_lo, d.batch, d.seq, 3 * GD, kGaBM, 64);
  if (rc) return rc;
  GateAttnArgs a;
  a.H = hcat;
  a.n = d.seq; a.n_qtiles = (d.seq + kGaBM - 1) / kGaBM;
  a.gate_heads = d.gate_heads; a.problems = d.batch * d.gate_heads; a.GD = GD; a.causal = d.gate_causal;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)kGaD));
  AG_CUDA_TRY(cudaFuncSetAttribute(gate_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGaSmemBytes));
  gate_attn_tc_kernel<<<a.n_qtiles * a.problems, kGaThreads, kGaSmemBytes, st>>>(tmHi, tmLo, a);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int gate_attn_tc_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
