// Prefill attention under the eviction mask (Eq. 2 with M_i of Eq. 5) on the
// Blackwell tensor cores, bf16, head_dim 128.
//
// One CTA handles 128 consecutive queries of one slab s = (sequence, head).
// Query j attends to cache rows r < prefix[s, j] (exactly the retained tokens
// before j, Sec. 3.3) and to itself (the diagonal of Eq. 5, always kept).  Over
// the compacted rows the mask is a staircase, so only the tiles that touch it
// need per-element masking and evicted keys are never loaded.
//
//   warp 0      TMA: Q tile once, then K / V tiles of 128 cache rows
//   warp 1      owns tensor memory, issues S = Q K^T (tcgen05.mma, operands in
//               shared memory) and O += P V (P read from tensor memory)
//   warps 2..5  one query row per thread: online softmax on S read from TMEM,
//               P written back to TMEM as bf16, O rescaled only when the running
//               maximum grows by more than 2^8, final normalisation and store
//
// TMEM columns: S [0,128), overwritten in place by P [0,64) (bf16 pairs); O [128,256).
// The self term seeds the running softmax (m = s_jj, l = 1) and its value row
// is added in the epilogue: O_j = (sum_r p_r v_r + w_self v_j) / l.
#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;

constexpr int kPfThreads = 192;
constexpr int kPfBM = 128, kPfBN = 128, kPfD = 128;
constexpr int kPfPanel = 128 * 128;                   // [128 rows][64 bf16] = 16 KB
constexpr int kPfTile = 2 * kPfPanel;                 // 32 KB
constexpr int kPfSmemBytes = 3 * kPfTile + 1024 + 256;
constexpr uint32_t kColS = 0, kColP = 0, kColO = 128, kTmemCols = 256;
constexpr float kRescaleThreshold = 8.f;              // log2 units

struct PrefillTcArgs {
  const __nv_bfloat16 *Q, *K, *V;   // dense [slabs, n, 128]
  __nv_bfloat16 *O;
  const int32_t *prefix;            // [slabs, n + 1]
  const int64_t *row_off;
  const int32_t *len;
  int n, n_qtiles, slabs;
  float scale_log2;
};

// Two CTAs share an SM (256 TMEM columns, 97 KB of shared memory each): inside a
// CTA the chain S = Q K^T -> softmax -> O += P V is serial, and the tensor core
// works on one CTA's tile while the other CTA is in its softmax.
__global__ void __launch_bounds__(kPfThreads, 2)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const PrefillTcArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t *sQ = smem;
  uint8_t *sK = sQ + kPfTile;
  uint8_t *sV = sK + kPfTile;
  uint64_t *bars = reinterpret_cast<uint64_t *>(sV + kPfTile);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 2, *v_full = bars + 3, *v_empty = bars + 4;
  uint64_t *s_full = bars + 5, *p_ready = bars + 6, *pv_done = bars + 7;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // heaviest query tiles first
  const int qt = a.n_qtiles - 1 - (int)(blockIdx.x / a.slabs);
  const int slab = blockIdx.x % a.slabs;
  const int j0 = qt * kPfBM;
  const int j_last = min(j0 + kPfBM, a.n) - 1;
  const int32_t *pre = a.prefix + (size_t)slab * (a.n + 1);
  const int max_bound = pre[j_last];               // keys any row of this tile may see
  const int n_kv = (max_bound + kPfBN - 1) / kPfBN;
  const int row0 = (int)a.row_off[slab];

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(k_full, 1); mbar_init(k_empty, 1);
    mbar_init(v_full, 1); mbar_init(v_empty, 1);
    mbar_init(s_full, 1);
    mbar_init(p_ready, 128);
    mbar_init(pv_done, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmQ); prefetch_tensormap(&tmK); prefetch_tensormap(&tmV);
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
    if (lane == 0 && n_kv > 0) {
      mbar_arrive_expect_tx(q_full, kPfTile);
      tma_load_3d(sQ, &tmQ, q_full, 0, j0, slab);
      tma_load_3d(sQ + kPfPanel, &tmQ, q_full, 64, j0, slab);
      for (int i = 0; i < n_kv; ++i) {
        const uint32_t ph = i & 1;
        const int y = row0 + i * kPfBN;
        if (!mbar_wait(k_empty, ph ^ 1)) break;
        mbar_arrive_expect_tx(k_full, kPfTile);
        tma_load_2d(sK, &tmK, k_full, 0, y);
        tma_load_2d(sK + kPfPanel, &tmK, k_full, 64, y);
        if (!mbar_wait(v_empty, ph ^ 1)) break;
        mbar_arrive_expect_tx(v_full, kPfTile);
        tma_load_2d(sV, &tmV, v_full, 0, y);
        tma_load_2d(sV + kPfPanel, &tmV, v_full, 64, y);
      }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------- MMA issuer
    if (lane == 0 && n_kv > 0) {
      const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
      bool ok = mbar_wait(q_full, 0);
      for (int i = 0; i < n_kv && ok; ++i) {
        const uint32_t ph = i & 1;
        // keys of this tile any row can see, rounded up to the MMA's N / K granularity
        const int keys = min(kPfBN, (max_bound - i * kPfBN + 15) & ~15);
        const uint32_t idesc_qk = idesc_bf16_f32(kPfBM, keys, false, false);
        constexpr uint32_t idesc_pv = idesc_bf16_f32(kPfBM, kPfD, false, true);
        if (!mbar_wait(k_full, ph)) { ok = false; break; }
        tc_fence_after_sync();
#pragma unroll
        for (int k = 0; k < kPfD / 16; ++k) {
          const uint32_t off = (k >> 2) * kPfPanel + (k & 3) * 32;
          mma_ss(tmem + kColS, desc_kmajor_sw128(q_addr + off), desc_kmajor_sw128(k_addr + off), idesc_qk, k != 0);
        }
        mma_commit(k_empty);
        mma_commit(s_full);
        if (!mbar_wait(p_ready, ph)) { ok = false; break; }
        if (!mbar_wait(v_full, ph)) { ok = false; break; }
        tc_fence_after_sync();
        for (int k = 0; k < keys / 16; ++k)
          mma_ts(tmem + kColO, tmem + kColP + k * 8, desc_mnmajor_sw128(v_addr + k * 2048, kPfPanel), idesc_pv,
                 (i | k) != 0);
        mma_commit(v_empty);
        mma_commit(pv_done);
        // P lives in the columns the next Q K^T overwrites, and the softmax threads
        // rescale O between tiles: let this P V finish first
        if (i + 1 < n_kv && !mbar_wait(pv_done, ph)) { ok = false; break; }
      }
    }
  } else {
    // ------------------------------------------- softmax / correction / epilogue
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may access
    const int row = quad * 32 + lane;
    const int j = j0 + row;
    const bool valid = j < a.n;
    const int jc = min(j, a.n - 1);
    const int bound = valid ? pre[jc] : 0;
    const int L = a.len[slab];
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const size_t row_elem = ((size_t)slab * a.n + jc) * kPfD;

    // self term: q_j . k_j
    float s_self = 0.f;
    {
      const __nv_bfloat16 *qp = a.Q + row_elem, *kp = a.K + row_elem;
#pragma unroll 4
      for (int c = 0; c < kPfD / 8; ++c) {
        float qf[8], kf[8];
        Elem<__nv_bfloat16>::unpack(ldg128(qp + c * 8), qf);
        Elem<__nv_bfloat16>::unpack(ldg128(kp + c * 8), kf);
#pragma unroll
        for (int e = 0; e < 8; ++e) s_self = fmaf(qf[e], kf[e], s_self);
      }
    }
    const float self2 = s_self * a.scale_log2;
    float m = self2, l = 1.f;
    bool ok = true;

    for (int i = 0; i < n_kv && ok; ++i) {
      const uint32_t ph = i & 1;
      ok = mbar_wait(s_full, ph);
      if (!ok) break;
      tc_fence_after_sync();
      const int nvalid = min(max(bound - i * kPfBN, 0), kPfBN);
      const bool full = nvalid >= kPfBN;

      uint32_t r[128];
      tmem_ld_x128_sync(tm_lane + kColS, r);
      float tmax = -INFINITY;
      if (full) {
#pragma unroll
        for (int e = 0; e < 128; ++e) tmax = fmaxf(tmax, __uint_as_float(r[e]));
      } else {
#pragma unroll
        for (int e = 0; e < 128; ++e) {
          if (e >= nvalid) r[e] = 0xff800000u;        // -inf: weight 0 below
          tmax = fmaxf(tmax, __uint_as_float(r[e]));
        }
      }
      tmax *= a.scale_log2;                           // scale > 0: max commutes; -inf stays -inf
      float m_new;
      if (i == 0) m_new = fmaxf(m, tmax);
      else m_new = (tmax > m + kRescaleThreshold) ? tmax : m;
      const bool rescale = (i > 0) && __any_sync(0xffffffffu, m_new != m);
      const float alpha = fast_exp2(m - m_new);
      l *= alpha;

      // O is stable here: the previous P V completed before this tile's Q K^T was issued
      if (rescale) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld_x32_sync(tm_lane + kColO + c * 32, o);
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st_x32(tm_lane + kColO + c * 32, o);
        }
      }

      // p = 2^(s - m) as bf16 pairs, written over the columns S occupied
      float rowsum = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const float p0 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e]), a.scale_log2, -m_new));
          const float p1 = fast_exp2(fmaf(__uint_as_float(r[c * 16 + e + 1]), a.scale_log2, -m_new));
          rowsum += p0 + p1;
          pk[e >> 1] = pack_bf16x2(p0, p1);
        }
        tmem_st_x8(tm_lane + kColP + c * 8, pk);
      }
      l += rowsum;
      m = m_new;

      // Rows of the V tile past the slab's valid length hold whatever the pool
      // holds (possibly NaN bit patterns): their weight is 0, but 0 * NaN is NaN
      // in the tensor core, so zero them in shared memory before P V reads them.
      if ((i + 1) * kPfBN > L) {
        ok = mbar_wait(v_full, ph);
        if (!ok) break;
        if (i * kPfBN + row >= L) {
          uint4 z = make_uint4(0, 0, 0, 0);
          uint8_t *v0 = sV + row * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            *reinterpret_cast<uint4 *>(v0 + c * 16) = z;
            *reinterpret_cast<uint4 *>(v0 + kPfPanel + c * 16) = z;
          }
        }
        fence_proxy_async_smem();
      }
      tmem_st_wait();
      tc_fence_before_sync();
      mbar_arrive(p_ready);
    }

    // epilogue
    if (ok && n_kv > 0) {
      ok = mbar_wait(pv_done, (n_kv - 1) & 1);
      tc_fence_after_sync();
    }
    if (ok) {
      const float w_self = fast_exp2(self2 - m);
      const float inv = 1.f / l;
      const __nv_bfloat16 *vp = a.V + row_elem;
      __nv_bfloat16 *op = a.O + row_elem;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        if (n_kv > 0) {
          tmem_ld_x32_sync(tm_lane + kColO + c * 32, r);
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) r[e] = 0u;
        }
        if (valid) {
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float vf[8];
            Elem<__nv_bfloat16>::unpack(ldg128(vp + c * 32 + g * 8), vf);
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              const float x0 = fmaf(w_self, vf[e], __uint_as_float(r[g * 8 + e])) * inv;
              const float x1 = fmaf(w_self, vf[e + 1], __uint_as_float(r[g * 8 + e + 1])) * inv;
              o[e >> 1] = pack_bf16x2(x0, x1);
            }
            *reinterpret_cast<uint4 *>(op + c * 32 + g * 8) = make_uint4(o[0], o[1], o[2], o[3]);
          }
        }
      }
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
                      const int32_t *prefix, float scale, void *O, cudaStream_t st) {
  const int slabs = d.batch * d.heads;
  CUtensorMap tmQ, tmK, tmV;
  int rc = make_tmap_3d_bf16(&tmQ, Q, slabs, d.seq, kPfD, kPfBM, 64);
  if (rc) return rc;
  // an empty pool still needs a valid map: describe one row of the dense K / V instead (never read)
  const bool empty = c.pool_rows == 0;
  rc = make_tmap_2d_bf16(&tmK, empty ? K : c.k_rows, empty ? 1 : (uint64_t)c.pool_rows, kPfD, kPfD * 2, kPfBN, 64);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmV, empty ? V : c.v_rows, empty ? 1 : (uint64_t)c.pool_rows, kPfD, kPfD * 2, kPfBN, 64);
  if (rc) return rc;
  PrefillTcArgs a;
  a.Q = static_cast<const __nv_bfloat16 *>(Q);
  a.K = static_cast<const __nv_bfloat16 *>(K);
  a.V = static_cast<const __nv_bfloat16 *>(V);
  a.O = static_cast<__nv_bfloat16 *>(O);
  a.prefix = prefix; a.row_off = c.row_off; a.len = c.len;
  a.n = d.seq; a.n_qtiles = (d.seq + kPfBM - 1) / kPfBM; a.slabs = slabs;
  a.scale_log2 = scale * 1.4426950408889634f;
  AG_CUDA_TRY(cudaFuncSetAttribute(prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPfSmemBytes));
  prefill_tc_kernel<<<a.n_qtiles * slabs, kPfThreads, kPfSmemBytes, st>>>(tmQ, tmK, tmV, a);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int prefill_tc_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
