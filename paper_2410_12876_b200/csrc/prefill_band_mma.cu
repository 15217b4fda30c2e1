// Band pass of prefill attention under a recent-token window (Appendix, Table 6), bf16, head_dim 128.
//
// After the attention kernel, row j of O holds the softmax over the retained tokens before j and j
// itself, and lse[j] its log-sum-exp.  The window adds the EVICTED tokens among the w - 1 before j:
//   O_j <- (2^(lse - M) O_j + sum_t 2^(s_t - M) v_t) / (2^(lse - M) + sum_t 2^(s_t - M)),
//   s_t = scale * q_j . k_t,  M = max(lse, max_t s_t).
// Per 16 queries that is S = Q K^T against the 32 tokens that cover all their windows (w - 1 <= 16)
// and O_band = P V: two small dense contractions, done with warp-level m16n8k16 MMAs.  One CTA =
// 64 consecutive queries of one slab; their Q rows, O rows and the 80 dense K, V rows [j0 - 16,
// j0 + 64) go to shared memory by 16-byte asynchronous copies, each warp works on its 16 queries,
// and the O tile goes back with coalesced 16-byte stores.  A row with no evicted token in its window
// comes out bit-identical (weight 1, nothing added).
#include "ag_common.cuh"
#include "mma_sync.cuh"

namespace ag {

constexpr int kBmD = 128, kBmQ = 64, kBmHalo = 16, kBmKeys = kBmQ + kBmHalo;
constexpr int kBmThreads = 128;
constexpr int kBmSmemBytes = (2 * kBmQ + 2 * kBmKeys) * 256;   // Q, O, K, V tiles: 72 KB

__global__ void __launch_bounds__(kBmThreads, 3)
prefill_band_mma_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K,
                        const __nv_bfloat16 *__restrict__ V, const uint8_t *__restrict__ flags,
                        const float *__restrict__ lse, __nv_bfloat16 *__restrict__ O, int n, int heads,
                        int kv_heads, int R, float scale_log2) {
  extern __shared__ __align__(128) uint8_t bm_smem[];
  const int slab = blockIdx.y, j0 = blockIdx.x * kBmQ;
  const int kv = (slab / heads) * kv_heads + (slab % heads) / (heads / kv_heads);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const uint32_t sQ = (uint32_t)__cvta_generic_to_shared(bm_smem), sO = sQ + kBmQ * 256;
  const uint32_t sK = sO + kBmQ * 256, sV = sK + kBmKeys * 256;
  uint8_t *smO = bm_smem + kBmQ * 256;
  const uint8_t *Qg = reinterpret_cast<const uint8_t *>(Q) + (size_t)slab * n * 256;
  uint8_t *Og = reinterpret_cast<uint8_t *>(O) + (size_t)slab * n * 256;
  const uint8_t *Kg = reinterpret_cast<const uint8_t *>(K) + (size_t)kv * n * 256;
  const uint8_t *Vg = reinterpret_cast<const uint8_t *>(V) + (size_t)kv * n * 256;

  // rows outside [0, n) are clamped for the copy; they are masked (keys) or never stored (queries)
  for (int idx = threadIdx.x; idx < kBmQ * 16; idx += kBmThreads) {
    const int r = idx >> 4, c = idx & 15;
    const size_t src = (size_t)min(j0 + r, n - 1) * 256 + c * 16;
    cp_async16(sQ + tile256_off(r, c), Qg + src);
    cp_async16(sO + tile256_off(r, c), Og + src);
  }
  for (int idx = threadIdx.x; idx < kBmKeys * 16; idx += kBmThreads) {
    const int r = idx >> 4, c = idx & 15;
    const size_t src = (size_t)min(max(j0 - kBmHalo + r, 0), n - 1) * 256 + c * 16;
    cp_async16(sK + tile256_off(r, c), Kg + src);
    cp_async16(sV + tile256_off(r, c), Vg + src);
  }
  cp_async_commit();

  // the warp's 32 key rows [16 warp, 16 warp + 32) of the key tile: bit l set = token evicted
  const int tok0 = j0 - kBmHalo + warp * 16;                    // token of the warp's key row 0
  const int my_tok = tok0 + lane;
  const bool ev = my_tok >= 0 && my_tok < n && flags[(size_t)kv * n + min(max(my_tok, 0), n - 1)] == 0;
  const uint32_t evicted = __ballot_sync(0xffffffffu, ev);
  float row_lse[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) row_lse[h] = lse[(size_t)slab * n + min(j0 + warp * 16 + g + 8 * h, n - 1)];

  cp_async_wait<0>();
  __syncthreads();

  // S = Q K^T: 16 queries x 32 keys
  float s[4][4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) s[nt][e] = 0.f;
#pragma unroll
  for (int ks = 0; ks < kBmD / 16; ++ks) {
    const int mi = lane >> 3;
    uint32_t a[4], b[4];
    // A: (rows 0-7, dims lo), (rows 8-15, dims lo), (rows 0-7, dims hi), (rows 8-15, dims hi)
    ldmatrix_x4(a, sQ + tile256_off(warp * 16 + (mi & 1) * 8 + (lane & 7), ks * 2 + (mi >> 1)));
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      // B: (keys 0-7, dims lo), (keys 0-7, dims hi), (keys 8-15, dims lo), (keys 8-15, dims hi) of this half
      ldmatrix_x4(b, sK + tile256_off(warp * 16 + half * 16 + (mi >> 1) * 8 + (lane & 7), ks * 2 + (mi & 1)));
      mma_16816(s[2 * half], a, b[0], b[1]);
      mma_16816(s[2 * half + 1], a, b[2], b[3]);
    }
  }

  // extend each row's softmax: key row kr of the warp is token tok0 + kr, query row r is token tok0 + 16 + r
  uint32_t pa[2][4];
  float w0[2], inv[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = g + 8 * h;
    const bool row_ok = j0 + warp * 16 + r < n;
    float sc[8], self = 0.f, smax = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int kr = nt * 8 + 2 * t + e;
        const int back = 16 + r - kr;                           // how far behind the query the key is
        const float v = s[nt][2 * h + e] * scale_log2;
        if (back == 0) self = v;
        const bool in = row_ok && back >= 1 && back <= R && ((evicted >> kr) & 1u);
        sc[nt * 2 + e] = in ? v : -INFINITY;
        smax = fmaxf(smax, sc[nt * 2 + e]);
      }
    self += __shfl_xor_sync(0xffffffffu, self, 1);
    self += __shfl_xor_sync(0xffffffffu, self, 2);
    smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 1));
    smax = fmaxf(smax, __shfl_xor_sync(0xffffffffu, smax, 2));
    // a tile whose queries had no retained key left O_j = v_j and no log-sum-exp: it is the self score
    const float base = row_lse[h] == -INFINITY ? self : row_lse[h];
    const float M = fmaxf(base, smax);
    float p[8], lsum = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      p[e] = exp2f(sc[e] - M);                                  // 0 for masked entries
      lsum += p[e];
    }
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
    lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
    w0[h] = exp2f(base - M);
    inv[h] = 1.f / (w0[h] + lsum);
    // A fragments of P for the two 16-key steps
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
      pa[kk][h] = pack2_bf16(p[kk * 4 + 0], p[kk * 4 + 1]);
      pa[kk][2 + h] = pack2_bf16(p[kk * 4 + 2], p[kk * 4 + 3]);
    }
  }

  // O_band = P V and the merge with the O tile, two 8-dim column tiles at a time
#pragma unroll
  for (int nt2 = 0; nt2 < kBmD / 16; ++nt2) {
    float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
      uint32_t b[4];
      // (keys 0-7, dims lo), (keys 8-15, dims lo), (keys 0-7, dims hi), (keys 8-15, dims hi) of this step
      const int mi = lane >> 3, row = warp * 16 + kk * 16 + (mi & 1) * 8 + (lane & 7);
      ldmatrix_x4_trans(b, sV + tile256_off(row, nt2 * 2 + (mi >> 1)));
      mma_16816(o0, pa[kk], b[0], b[1]);
      mma_16816(o1, pa[kk], b[2], b[3]);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int row = warp * 16 + g + 8 * h;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        // dims 16 nt2 + 8 half + 2t, +1 of this row: one 32-bit word of the O tile
        uint32_t *w = reinterpret_cast<uint32_t *>(smO + tile256_off(row, nt2 * 2 + half) + t * 4);
        const __nv_bfloat162 old = *reinterpret_cast<__nv_bfloat162 *>(w);
        const float *ob = half == 0 ? o0 : o1;
        const float x0 = fmaf(w0[h], __low2float(old), ob[2 * h]) * inv[h];
        const float x1 = fmaf(w0[h], __high2float(old), ob[2 * h + 1]) * inv[h];
        *w = pack2_bf16(x0, x1);
      }
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < kBmQ * 16; idx += kBmThreads) {
    const int r = idx >> 4, c = idx & 15;
    if (j0 + r < n)
      *reinterpret_cast<uint4 *>(Og + (size_t)(j0 + r) * 256 + c * 16) =
          *reinterpret_cast<const uint4 *>(smO + tile256_off(r, c));
  }
}

int launch_prefill_band_mma(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                            const uint8_t *flags, const float *lse, float scale, void *O, cudaStream_t st) {
  AG_CUDA_TRY(cudaFuncSetAttribute(prefill_band_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   kBmSmemBytes));
  dim3 grid((d.seq + kBmQ - 1) / kBmQ, d.batch * d.heads);
  prefill_band_mma_kernel<<<grid, kBmThreads, kBmSmemBytes, st>>>(
      static_cast<const __nv_bfloat16 *>(Q), static_cast<const __nv_bfloat16 *>(K),
      static_cast<const __nv_bfloat16 *>(V), flags, lse, static_cast<__nv_bfloat16 *>(O), d.seq, d.heads,
      kv_heads_of(d), recent_rows(d), scale * 1.4426950408889634f);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace ag
