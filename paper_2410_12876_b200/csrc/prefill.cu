// Prefill attention under the eviction mask (Eq. 2 with the mask M_i of Eq. 5).
//
// Query j of slab s = (sequence, head) sees the retained tokens before it and
// itself.  The retained tokens before j are exactly rows r < prefix[s, j] of
// the compacted cache, so the mask of Eq. 5 becomes a monotone staircase over
// contiguous cache rows; the self term comes from the dense K, V.
#include "ag_common.cuh"
#include "attn_simt.cuh"

namespace ag {

size_t prefill_workspace_bytes(const ag_layer_desc &) { return 0; }

template <typename T, int D>
static int run_prefill_simt(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                            const ag_cache &c, const int32_t *prefix, float scale, void *O,
                            cudaStream_t st) {
  SimtAttnArgs a{};
  a.Q = Q; a.K = K; a.V = V; a.O = O;
  a.n = d.seq; a.inner = d.heads; a.kv_group = d.heads / kv_heads_of(d);
  const long long head = (long long)d.seq * D, batch = head * d.heads;
  a.q_batch = a.o_batch = batch;
  a.k_batch = a.v_batch = head * kv_heads_of(d);
  a.q_inner = a.k_inner = a.v_inner = a.o_inner = head;
  a.q_row = a.k_row = a.v_row = a.o_row = D;
  a.scale_log2 = scale * 1.4426950408889634f;
  a.k_rows = c.k_rows; a.v_rows = c.v_rows; a.row_off = c.row_off; a.prefix = prefix;
  return launch_simt_attn<T, T, D, kPrefill>(a, d.batch * d.heads, st);
}

int launch_prefill(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                   const uint8_t *, const ag_cache &c, const int32_t *prefix, float scale,
                   void *O, void *, cudaStream_t st) {
  if (prefill_tc_supported(d, c)) return launch_prefill_tc(d, Q, K, V, c, prefix, scale, O, st);
  if (d.dtype == AG_F32) {
    if (d.head_dim == 64) return run_prefill_simt<float, 64>(d, Q, K, V, c, prefix, scale, O, st);
    return run_prefill_simt<float, 128>(d, Q, K, V, c, prefix, scale, O, st);
  }
  if (d.head_dim == 64) return run_prefill_simt<__nv_bfloat16, 64>(d, Q, K, V, c, prefix, scale, O, st);
  return run_prefill_simt<__nv_bfloat16, 128>(d, Q, K, V, c, prefix, scale, O, st);
}

}  // namespace ag
