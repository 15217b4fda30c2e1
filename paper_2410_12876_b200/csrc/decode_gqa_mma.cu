// Chunk pass of decode attention for grouped-query attention on the tensor cores.
//
// The G query heads that share a key/value head meet the same rows of the slab, so one step of the
// decoding stage (Sec. 3.1) is, per slab, the small dense contraction S = Q_g K^T (G x L x D) and
// O = P V (G x D x L), not G matrix-vector products.  On CUDA cores that costs G dot products and G
// weighted sums per row and the kernel ends up bound by arithmetic, not by HBM; decode_mma_core.cuh
// runs it on warp-level MMAs.  One CTA = one chunk of one key/value slab, as in the CUDA-core chunk
// pass; it leaves one (m, l, o) triple per query head of the group where decode_combine_kernel
// expects it.
#include "decode_mma_core.cuh"

namespace ag {

// two stages x three CTAs per SM measured better here than deeper rings in fewer CTAs
constexpr int kGqChunkStages = 2;
__global__ void __launch_bounds__(kGqThreads, 3)
decode_partial_gqa_mma_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_rows,
                              const __nv_bfloat16 *__restrict__ v_rows, const int64_t *__restrict__ row_off,
                              const int32_t *__restrict__ len, float scale_log2, int chunk_rows,
                              float *__restrict__ part_o, float *__restrict__ part_ml, int kv_heads, int G,
                              int max_splits) {
  extern __shared__ __align__(128) uint8_t gq_smem[];
  const int kv = blockIdx.y, chunk = blockIdx.x;
  const int slab0 = (kv / kv_heads) * kv_heads * G + (kv % kv_heads) * G;     // first query slab of the group
  const int L = len[kv];
  const int r_begin = chunk * chunk_rows;
  if (r_begin >= L) return;                                                    // the whole CTA, before any barrier
  const int r_end = min(L, r_begin + chunk_rows);
  const uint8_t *Kg = reinterpret_cast<const uint8_t *>(k_rows) + (size_t)row_off[kv] * kGqRowBytes;
  const uint8_t *Vg = reinterpret_cast<const uint8_t *>(v_rows) + (size_t)row_off[kv] * kGqRowBytes;
  const GqWarpTriples w = gq_stream_rows<kGqChunkStages>(gq_smem, q + (size_t)slab0 * kGqD, G, Kg, Vg, r_begin, r_end, scale_log2);
  for (int x = threadIdx.x; x < G * kGqD; x += kGqThreads) {     // one (head, output dimension) at a time
    const int h = x / kGqD, d = x % kGqD;
    float acc, mc, lc;
    gq_combine(w, h, d, acc, mc, lc);
    const size_t slot = (size_t)(slab0 + h) * max_splits + chunk;
    part_o[slot * kGqD + d] = acc;
    if (d == 0) {
      part_ml[slot * 2 + 0] = mc;
      part_ml[slot * 2 + 1] = lc;
    }
  }
}

bool decode_gqa_mma_supported(const ag_layer_desc &d) {
  const int group = d.heads / kv_heads_of(d);
  return d.dtype == AG_BF16 && d.head_dim == kGqD && group >= 2 && group <= kGqMaxGroup;
}

int launch_decode_partial_gqa_mma(const ag_layer_desc &d, const void *q, const ag_cache &c, float scale_log2,
                                  int chunk_rows, int n_chunks, float *part_o, float *part_ml, int max_splits,
                                  cudaStream_t st) {
  const int kvh = kv_heads_of(d);
  AG_CUDA_TRY(cudaFuncSetAttribute(decode_partial_gqa_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   gq_smem_bytes(kGqChunkStages)));
  dim3 grid(n_chunks, d.batch * kvh);
  decode_partial_gqa_mma_kernel<<<grid, kGqThreads, gq_smem_bytes(kGqChunkStages), st>>>(
      static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(c.k_rows),
      static_cast<const __nv_bfloat16 *>(c.v_rows), c.row_off, c.len, scale_log2, chunk_rows, part_o, part_ml,
      kvh, d.heads / kvh, max_splits);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace ag
