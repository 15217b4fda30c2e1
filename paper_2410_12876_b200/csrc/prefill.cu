// Prefill attention under the eviction mask (Eq. 2 with the mask M_i of Eq. 5).
//
// Query j of slab s = (sequence, head) sees the retained tokens before it and
// itself.  The retained tokens before j are exactly rows r < prefix[s, j] of
// the compacted cache, so the mask of Eq. 5 becomes a monotone staircase over
// contiguous cache rows; the self term comes from the dense K, V.
#include "ag_common.cuh"
#include "attn_simt.cuh"

namespace ag {

// With a recent-token window the attention kernels leave each row's log-sum-exp in the workspace
// for the band pass below.
size_t prefill_workspace_bytes(const ag_layer_desc &d) {
  if (recent_rows(d) == 0) return 0;
  return align_up((size_t)d.batch * d.heads * d.seq * sizeof(float), 256);
}

// Recent-token window (Appendix, Table 6): query j also sees the EVICTED tokens among the
// w - 1 before it (the retained ones and j itself are in O already).  One lane group per query:
// scores of those tokens against the dense K, then the row's softmax is extended by them,
//   O_j <- (2^(lse - M) O_j + sum_t 2^(s_t - M) v_t) / (2^(lse - M) + sum_t 2^(s_t - M)),
// with lse the row's log-sum-exp from the attention kernel and M the larger of lse and max s_t.
// Rows with no evicted token in their window are left untouched.  CUDA-core form, for fp32 and
// head_dim 64; bf16 with head_dim 128 takes prefill_band_mma_kernel.
constexpr int kBandThreads = 256;
template <typename T, int D>
__global__ void __launch_bounds__(kBandThreads)
prefill_band_kernel(const T *__restrict__ Q, const T *__restrict__ K, const T *__restrict__ V,
                    const uint8_t *__restrict__ flags, const float *__restrict__ lse, T *__restrict__ O,
                    int n, int heads, int kv_heads, int R, float scale_log2) {
  constexpr int kEpl = Elem<T>::kPerVec;
  constexpr int kLanes = D / kEpl;                 // lanes per query
  constexpr int kRowsPerCta = kBandThreads / kLanes;
  const int slab = blockIdx.y;
  const int kv = (slab / heads) * kv_heads + (slab % heads) / (heads / kv_heads);
  const int g = threadIdx.x / kLanes, v = threadIdx.x % kLanes;
  const int j = min(blockIdx.x * kRowsPerCta + g, n - 1);     // clamped rows recompute row n - 1, store nothing
  const bool valid = blockIdx.x * kRowsPerCta + g < n;
  const uint8_t *f = flags + (size_t)kv * n;
  const T *Kd = K + (size_t)kv * n * D + v * kEpl;
  const T *Vd = V + (size_t)kv * n * D + v * kEpl;

  float qf[kEpl];
  Elem<T>::unpack(ldg128(Q + ((size_t)slab * n + j) * D + v * kEpl), qf);
#pragma unroll
  for (int e = 0; e < kEpl; ++e) qf[e] *= scale_log2;

  // scores of the evicted tokens of the window; every lane of the group ends with the same values
  float s[kMaxRecent];
  float smax = -INFINITY;
#pragma unroll
  for (int u = 0; u < kMaxRecent; ++u) {
    if (u >= R) {                                    // the same for the whole grid
      s[u] = -INFINITY;
      continue;
    }
    const int t = j - 1 - u;
    const bool in = t >= 0 && f[max(t, 0)] == 0;
    float kf[kEpl];
    Elem<T>::unpack(ldg128(Kd + (size_t)max(t, 0) * D), kf);
    float a = 0.f;
#pragma unroll
    for (int e = 0; e < kEpl; ++e) a = fmaf(qf[e], kf[e], a);
#pragma unroll
    for (int off = kLanes / 2; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
    s[u] = in ? a : -INFINITY;
    smax = fmaxf(smax, s[u]);
  }
  if (smax == -INFINITY || !valid) return;           // no shuffles below: lanes may leave

  float row_lse = lse[(size_t)slab * n + j];
  if (row_lse == -INFINITY) {
    // the attention kernel skipped the scores of this tile (no retained key): O_j = v_j, weight 2^(q_j . k_j)
    float kf[kEpl];
    Elem<T>::unpack(ldg128(Kd + (size_t)j * D), kf);
    float a = 0.f;
#pragma unroll
    for (int e = 0; e < kEpl; ++e) a = fmaf(qf[e], kf[e], a);
    // the lanes of a group are still together here (the early return above is uniform per group),
    // but other groups of the warp may have left: reduce through the group's own lanes only
    const unsigned lane = threadIdx.x & 31u;
    const unsigned group_mask = kLanes == 32 ? 0xffffffffu : (((1u << kLanes) - 1u) << (lane / kLanes * kLanes));
#pragma unroll
    for (int off = kLanes / 2; off > 0; off >>= 1) a += __shfl_xor_sync(group_mask, a, off);
    row_lse = a;
  }
  const float M = fmaxf(row_lse, smax);
  const float w0 = exp2f(row_lse - M);
  float of[kEpl];
  T *Oj = O + ((size_t)slab * n + j) * D + v * kEpl;
  Elem<T>::unpack(ldg128(Oj), of);
  float lsum = w0;
#pragma unroll
  for (int e = 0; e < kEpl; ++e) of[e] *= w0;
#pragma unroll
  for (int u = 0; u < kMaxRecent; ++u) {
    if (s[u] == -INFINITY) continue;
    const float p = exp2f(s[u] - M);
    float vf[kEpl];
    Elem<T>::unpack(ldg128(Vd + (size_t)(j - 1 - u) * D), vf);
    lsum += p;
#pragma unroll
    for (int e = 0; e < kEpl; ++e) of[e] = fmaf(p, vf[e], of[e]);
  }
  const float inv = 1.f / lsum;
#pragma unroll
  for (int e = 0; e < kEpl; ++e) Elem<T>::store(Oj + e, of[e] * inv);
}

template <typename T, int D>
static int run_prefill_band(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                            const uint8_t *flags, const float *lse, float scale, void *O, cudaStream_t st) {
  constexpr int kRowsPerCta = kBandThreads / (D / Elem<T>::kPerVec);
  dim3 grid((d.seq + kRowsPerCta - 1) / kRowsPerCta, d.batch * d.heads);
  prefill_band_kernel<T, D><<<grid, kBandThreads, 0, st>>>(
      static_cast<const T *>(Q), static_cast<const T *>(K), static_cast<const T *>(V), flags, lse,
      static_cast<T *>(O), d.seq, d.heads, kv_heads_of(d), recent_rows(d), scale * 1.4426950408889634f);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

template <typename T, int D>
static int run_prefill_simt(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                            const ag_cache &c, const int32_t *prefix, float scale, void *O,
                            float *lse, cudaStream_t st) {
  SimtAttnArgs a{};
  a.Q = Q; a.K = K; a.V = V; a.O = O;
  a.n = d.seq; a.inner = d.heads; a.kv_group = d.heads / kv_heads_of(d);
  const long long head = (long long)d.seq * D, batch = head * d.heads;
  a.q_batch = a.o_batch = batch;
  a.k_batch = a.v_batch = head * kv_heads_of(d);
  a.q_inner = a.k_inner = a.v_inner = a.o_inner = head;
  a.q_row = a.k_row = a.v_row = a.o_row = D;
  a.scale_log2 = scale * 1.4426950408889634f;
  a.k_rows = c.k_rows; a.v_rows = c.v_rows; a.row_off = c.row_off; a.prefix = prefix; a.len = c.len;
  a.seq_lens = d.seq_lens;
  a.lse = lse;
  return launch_simt_attn<T, T, D, kPrefill>(a, d.batch * d.heads, st);
}

template <typename T, int D>
static int run_prefill(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                       const uint8_t *flags, const ag_cache &c, const int32_t *prefix, float scale,
                       void *O, float *lse, cudaStream_t st) {
  int rc = run_prefill_simt<T, D>(d, Q, K, V, c, prefix, scale, O, lse, st);
  if (rc || !lse) return rc;
  return run_prefill_band<T, D>(d, Q, K, V, flags, lse, scale, O, st);
}

int launch_prefill(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                   const uint8_t *flags, const ag_cache &c, const int32_t *prefix, float scale,
                   void *O, void *ws, cudaStream_t st) {
  float *lse = recent_rows(d) > 0 ? static_cast<float *>(ws) : nullptr;
  if (prefill_tc_supported(d, c)) {
    int rc = launch_prefill_tc(d, Q, K, V, c, prefix, scale, O, lse, st);
    if (rc || !lse) return rc;
    return launch_prefill_band_mma(d, Q, K, V, flags, lse, scale, O, st);
  }
  if (d.dtype == AG_F32) {
    if (d.head_dim == 64) return run_prefill<float, 64>(d, Q, K, V, flags, c, prefix, scale, O, lse, st);
    return run_prefill<float, 128>(d, Q, K, V, flags, c, prefix, scale, O, lse, st);
  }
  if (d.head_dim == 64) return run_prefill<__nv_bfloat16, 64>(d, Q, K, V, flags, c, prefix, scale, O, lse, st);
  int rc = run_prefill_simt<__nv_bfloat16, 128>(d, Q, K, V, c, prefix, scale, O, lse, st);
  if (rc || !lse) return rc;
  return launch_prefill_band_mma(d, Q, K, V, flags, lse, scale, O, st);
}

}  // namespace ag
