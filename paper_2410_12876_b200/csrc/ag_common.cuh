// Shared device/host helpers for the AG-gated attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ag.h"

namespace ag {

// ---------------------------------------------------------------- host side
void set_last_cuda_error(int e);

#define AG_CUDA_TRY(expr)                                 \
  do {                                                    \
    cudaError_t _e = (expr);                              \
    if (_e != cudaSuccess) {                              \
      ::ag::set_last_cuda_error((int)_e);                 \
      return AG_ERR_CUDA;                                 \
    }                                                     \
  } while (0)

#define AG_LAUNCH_CHECK() AG_CUDA_TRY(cudaGetLastError())

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// Key/value heads of the layer (grouped-query attention), = heads when the field is 0.
inline int kv_heads_of(const ag_layer_desc &d) { return d.kv_heads > 0 ? d.kv_heads : d.heads; }
// Launch attribute that lets a kernel overlap its set-up with the tail of its predecessor (the
// kernel itself starts with pdl_wait()).
inline cudaLaunchAttribute pdl_attribute() {
  cudaLaunchAttribute at = {};
  at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at.val.programmaticStreamSerializationAllowed = 1;
  return at;
}
// Recent-token window: the ring of a slab holds the last recent_window - 1 tokens (0 = no ring).
constexpr int kMaxRecent = 16;
inline int recent_rows(const ag_layer_desc &d) { return d.recent_window > 1 ? d.recent_window - 1 : 0; }
// The ring of a cache as the kernels take it (R = 0: the layer has no window, nothing is touched).
struct RecentRing {
  void *k, *v;        // [slabs, R, D]
  uint8_t *live;      // [slabs, R]
  int32_t *pos;       // [slabs]
  int R;
};
inline RecentRing ring_of(const ag_layer_desc &d, const ag_cache &c) {
  RecentRing r = {};
  r.R = recent_rows(d);
  if (r.R > 0) { r.k = c.recent_k; r.v = c.recent_v; r.live = c.recent_live; r.pos = c.pos; }
  return r;
}
inline bool misaligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Host-side argument checks shared by every entry point (ag_api.cu): the descriptor fields all calls
// use (sizes, dtype, head_dim, the key/value head grouping, the recent-token window) and the cache
// struct (need_recent: the call reads or writes the ring of recent tokens).
int check_desc(const ag_layer_desc *d);
int check_cache(const ag_cache *c, const ag_layer_desc *d = nullptr, bool need_recent = false);

// Per-step launchers (defined in the kernel files, called from ag_api.cu).
size_t gate_workspace_bytes(const ag_layer_desc &d);
int launch_gate(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk,
                const void *Wv, const void *Wo, const float *gamma, float *scores,
                uint8_t *flags, void *ws, cudaStream_t st);

// Tensor-core (tcgen05) projection GEMM for bf16 inputs: [M, 3*GD] = X [W0 | W1 | W2], written
// either as float32 (C) or, when Chi / Clo are given, as the bf16 pair hi + lo of each float32 value.
bool gate_proj_tc_supported(int K, int GD);
int launch_gate_proj_tc(const void *X, const void *W0, const void *W1, const void *W2, float *C, void *Chi,
                        void *Clo, int M, int K, int GD, cudaStream_t st);
// Tensor-core MHA' (Sec. 3.3) on the hi / lo pairs, then the split-K merge fused with the gate's
// output layer and threshold (Eq. 3, Eq. 4): scores (optional) and flags [B, h, n].
bool gate_attn_tc_supported(const ag_layer_desc &d);
size_t gate_attn_partial_bytes(const ag_layer_desc &d);   // split-K partials (workspace)
int launch_gate_attn_tc(const ag_layer_desc &d, const void *qkv_hi, const void *qkv_lo, void *partials,
                        const void *Wo, const float *gamma, float logit_tau, float *scores, uint8_t *flags,
                        cudaStream_t st);
int gate_attn_tc_wait_timeouts();
// The local gate of Sec. 3.4: s = X W_lin and the threshold of Eq. 4.
int launch_gate_linear(const ag_layer_desc &d, const void *X, const void *W, const float *gamma,
                       float *scores, uint8_t *flags, cudaStream_t st);
int gate_linear_wait_timeouts();
int gemm_tc_wait_timeouts();

size_t compact_workspace_bytes(const ag_layer_desc &d);
int launch_compact(const ag_layer_desc &d, const void *K, const void *V, const uint8_t *flags,
                   const ag_cache &c, int32_t *prefix, int32_t *idx, int32_t *dev_status,
                   void *ws, cudaStream_t st);

// Key/value projection (Eq. 2) on the tensor cores with the retained rows written straight into the
// ragged cache (bf16, head_dim 128).
bool kv_proj_cache_supported(const ag_layer_desc &d);
// Wq, Q: NULL, or the query projection Q = X Wq rides in the same launch (dense output only).
int launch_kv_proj_cache(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk, const void *Wv,
                         const uint8_t *flags, const ag_cache &c, int32_t *prefix, int32_t *idx, void *Q, void *K,
                         void *V, int32_t *dev_status, cudaStream_t st);
int kv_proj_cache_wait_timeouts();

// Fills the ring of a recent-token window (no-op without one) from the dense K, V of the prompt.
int launch_recent_fill(const ag_layer_desc &d, const void *K, const void *V, const uint8_t *flags, const ag_cache &c,
                       cudaStream_t st);

size_t prefill_workspace_bytes(const ag_layer_desc &d);
int launch_prefill(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                   const uint8_t *flags, const ag_cache &c, const int32_t *prefix, float scale,
                   void *O, void *ws, cudaStream_t st);

// Tensor-core (tcgen05) prefill attention for bf16, head_dim 128.
bool prefill_tc_supported(const ag_layer_desc &d, const ag_cache &c);
// lse (NULL or [slabs, n]): log2 of each row's softmax denominator, in the units of the scaled
// scores times log2(e); -inf where a whole query tile had no retained key (O = v_j there).
int launch_prefill_tc(const ag_layer_desc &d, const void *Q, const void *K, const void *V, const ag_cache &c,
                      const int32_t *prefix, float scale, void *O, float *lse, cudaStream_t st);
int prefill_tc_wait_timeouts();
// Band pass of a recent-token window on the tensor cores (bf16, head_dim 128): extends every row of O
// by the evicted tokens of its window, given the rows' log-sum-exp.
int launch_prefill_band_mma(const ag_layer_desc &d, const void *Q, const void *K, const void *V,
                            const uint8_t *flags, const float *lse, float scale, void *O, cudaStream_t st);

// Output projection of Eq. 1 with the skip connection: Y = X_res + [H_1 .. H_h] Wo (tensor cores for
// bf16, head_dim 128; CUDA cores otherwise).
int launch_out_proj(const ag_layer_desc &d, const void *O, const void *Wo, const void *X_res, void *Y, cudaStream_t st);
int out_proj_wait_timeouts();

size_t decode_workspace_bytes(const ag_layer_desc &d);
int launch_decode(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                  const ag_cache &c, float scale, void *o, void *ws, size_t ws_bytes,
                  cudaStream_t st);
int launch_decode_step(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                       const uint8_t *flag_new, const ag_cache &c, float scale, void *o,
                       int32_t *dev_status, void *ws, cudaStream_t st);
// Chunk pass of decode for grouped-query attention on the tensor cores (bf16, head_dim 128, groups
// of 2..16 query heads): writes the (m, l, o) triples of every (query slab, chunk).
bool decode_gqa_mma_supported(const ag_layer_desc &d);
int launch_decode_partial_gqa_mma(const ag_layer_desc &d, const void *q, const ag_cache &c, float scale_log2,
                                  int chunk_rows, int n_chunks, float *part_o, float *part_ml, int max_splits,
                                  cudaStream_t st);
int launch_append(const ag_layer_desc &d, const void *k_new, const void *v_new,
                  const uint8_t *flag_new, const ag_cache &c, int32_t *dev_status,
                  cudaStream_t st);

// -------------------------------------------------------------- device side
#ifdef __CUDACC__
template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;  // elements in a 16-byte vector
  __device__ static inline void unpack(const uint4 &v, float *f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static inline float load(const float *p) { return *p; }
  __device__ static inline void store(float *p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static inline void unpack(const uint4 &v, float *f) {
    // bf16 -> f32 is a 16-bit left shift
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
  }
  __device__ static inline float load(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
  __device__ static inline void store(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }
};

// Programmatic dependent launch, for the small kernels of a decode step that run back to back:
// a kernel launched with the stream-serialization attribute may be set up while its predecessor
// in the stream is still running.  It must call pdl_wait() before it touches global memory (the
// predecessor has then completed, its writes visible); pdl_launch_dependents() lets the successor's
// set-up begin.  Both are no-ops in a launch without the attribute.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Puts the new token of slab `slab` into its ring (recent-token window): slot = tokens seen % R,
// marked live iff the token is NOT kept (a kept one is a row of the slab).  Called by kVecs
// consecutive lanes of one warp (vec = 0 .. kVecs - 1, one 16-byte piece of the row each), after
// every read of the ring by this launch.
template <int kVecs>
__device__ __forceinline__ void ring_put(const RecentRing &rg, int slab, int vec, const uint8_t *k_row,
                                         const uint8_t *v_row, bool kept) {
  const unsigned lane = threadIdx.x & 31u;
  const unsigned mask = kVecs == 32 ? 0xffffffffu : (((1u << kVecs) - 1u) << (lane / kVecs * kVecs));
  const int p = rg.pos[slab];
  __syncwarp(mask);                                 // every lane has read pos before it moves
  const int slot = p % rg.R;
  const size_t dst = ((size_t)slab * rg.R + slot) * (kVecs * 16) + vec * 16;
  *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(rg.k) + dst) = *reinterpret_cast<const uint4 *>(k_row + vec * 16);
  *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(rg.v) + dst) = *reinterpret_cast<const uint4 *>(v_row + vec * 16);
  if (vec == 0) {
    rg.live[(size_t)slab * rg.R + slot] = kept ? 0 : 1;
    rg.pos[slab] = p + 1;
  }
}

__device__ __forceinline__ uint4 ldg128(const void *p) {
  return __ldg(reinterpret_cast<const uint4 *>(p));
}
// Streaming 16-byte load that does not allocate in L1 (data used once).
__device__ __forceinline__ uint4 ldg128_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
#endif  // __CUDACC__

}  // namespace ag
