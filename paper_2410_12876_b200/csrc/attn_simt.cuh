// float32 CUDA-core attention used where the tensor-core path does not apply:
// the fp32 layer (tcgen05 has no true-fp32 MMA) and the fp32 internals of the
// gate (MHA' of Sec. 3.3 evaluated on float32 Q', K', V').
//
// One CTA = 64 query rows x one problem (sequence, head); keys are visited in
// tiles of 64 with an online softmax.  Row j sees the first bound(j) rows of
// the key array, where bound is
//   kGateCausal : j + 1            (lower-triangular mask inside MHA')
//   kGateFull   : n                (every token sees the whole sequence)
//   kPrefill    : prefix[s, j]     (retained tokens before j, read from the
//                                   compacted cache) plus the self term (k_j,
//                                   v_j) from the dense K, V: Eq. 5.
#pragma once
#include "ag_common.cuh"

namespace ag {

enum SimtAttnMode { kGateCausal = 0, kGateFull = 1, kPrefill = 2 };

struct SimtAttnArgs {
  const void *Q, *K, *V;      // kPrefill: K, V are the DENSE tensors (self term)
  void *O;
  int n;                      // query rows per problem
  int inner;                  // problems per batch element (h' or h)
  int kv_group;               // kPrefill: query heads per key/value head (0 or 1 = one each)
  long long q_batch, q_inner, q_row;   // element strides
  long long k_batch, k_inner, k_row;   // gate: K/V rows inside the packed projection
  long long v_batch, v_inner, v_row;
  long long o_batch, o_inner, o_row;
  float scale_log2;
  // kPrefill only
  const void *k_rows, *v_rows;         // compacted cache pools
  const int64_t *row_off;
  const int32_t *prefix;               // [problems, n + 1]
  const int32_t *len;                  // [problems] valid rows of each slab: a row bound never exceeds it
  float *lse;                          // NULL, or [problems, n]: m + log2(l) of every row
  // [batch] tokens each sequence has (the rest is padding), or NULL = n: the keys of kGateFull, and
  // the query tiles kPrefill has to compute
  const int32_t *seq_lens;
};

constexpr int kSimtBM = 64, kSimtBN = 64, kSimtThreads = 256;

template <int D>
constexpr size_t simt_attn_smem_bytes() {
  return sizeof(float) * ((size_t)kSimtBM * D + (size_t)D * (kSimtBN + 4) + (size_t)kSimtBN * D +
                          (size_t)kSimtBM * (kSimtBN + 4));
}

template <typename TIn, typename TOut, int D, int MODE>
__global__ void __launch_bounds__(kSimtThreads)
simt_attn_kernel(const SimtAttnArgs a) {
  extern __shared__ __align__(16) float smem[];
  float *Qs = smem;                               // [BM][D]
  float *Kt = Qs + kSimtBM * D;                   // [D][BN + 4]  (transposed)
  float *Vs = Kt + D * (kSimtBN + 4);             // [BN][D]
  float *Ps = Vs + kSimtBN * D;                   // [BM][BN + 4]
  constexpr int KP = kSimtBN + 4;
  constexpr int kEpl = Elem<TIn>::kPerVec;
  constexpr int kVecPerRow = D / kEpl;
  constexpr int kOC = D / 64;                     // float4 column groups per thread

  const int prob = blockIdx.y;
  const int b = prob / a.inner, i = prob % a.inner;
  const int j0 = blockIdx.x * kSimtBM;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  const TIn *Qp = static_cast<const TIn *>(a.Q) + b * a.q_batch + i * a.q_inner;
  // grouped-query attention: query head i reads key/value head ik, cache slab prob_kv
  const int group = a.kv_group > 1 ? a.kv_group : 1;
  const int ik = i / group, prob_kv = b * (a.inner / group) + ik;
  const TIn *Kd = static_cast<const TIn *>(a.K) + b * a.k_batch + ik * a.k_inner;
  const TIn *Vd = static_cast<const TIn *>(a.V) + b * a.v_batch + ik * a.v_inner;
  const TIn *Kp = Kd, *Vp = Vd;
  long long kp_row = a.k_row, vp_row = a.v_row;
  if (MODE == kPrefill) {
    Kp = static_cast<const TIn *>(a.k_rows) + a.row_off[prob_kv] * (long long)D;
    Vp = static_cast<const TIn *>(a.v_rows) + a.row_off[prob_kv] * (long long)D;
    kp_row = D; vp_row = D;
  }
  const int32_t *pre = MODE == kPrefill ? a.prefix + (size_t)prob_kv * (a.n + 1) : nullptr;
  // a slab that overflowed at compaction holds no rows (len = 0) although its prefix counts are
  // full: its queries then see themselves only, and no read leaves the slab
  const int slab_len = MODE == kPrefill ? a.len[prob_kv] : 0;
  const int n_keys = (MODE == kGateFull && a.seq_lens) ? a.seq_lens[prob / a.inner] : a.n;
  // prefill: a query tile past its sequence's end holds padding only (outputs unspecified): nothing to do
  if (MODE == kPrefill && a.seq_lens && j0 >= a.seq_lens[prob / a.inner]) return;

  // Q tile -> shared (rows past n are clamped; they are never stored)
  for (int x = tid; x < kSimtBM * kVecPerRow; x += kSimtThreads) {
    const int r = x / kVecPerRow, c = x % kVecPerRow;
    const int j = min(j0 + r, a.n - 1);
    float f[kEpl];
    Elem<TIn>::unpack(ldg128(Qp + j * a.q_row + c * kEpl), f);
#pragma unroll
    for (int e = 0; e < kEpl; ++e) Qs[r * D + c * kEpl + e] = f[e];
  }

  int bound[4];
  bool valid[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    const int j = j0 + ty * 4 + r;
    valid[r] = j < a.n;
    const int jc = min(j, a.n - 1);
    bound[r] = MODE == kGateCausal ? jc + 1 : (MODE == kGateFull ? n_keys : min(pre[jc], slab_len));
    if (!valid[r]) bound[r] = 0;
  }
  const int j_last = min(j0 + kSimtBM, a.n) - 1;
  const int max_bound = MODE == kGateCausal ? j_last + 1 : (MODE == kGateFull ? n_keys : min(pre[j_last], slab_len));
  const int n_tiles = (max_bound + kSimtBN - 1) / kSimtBN;

  float m[4], l[4], o[4][kOC][4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
    for (int c = 0; c < kOC; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[r][c][e] = 0.f;
  }
  __syncthreads();

  if (MODE == kPrefill) {
    // self term: the diagonal of Eq. 5 seeds the running softmax (m = s_jj, l = 1, o = v_j)
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int row = ty * 4 + r;
      const int j = min(j0 + row, a.n - 1);
      float acc = 0.f;
      for (int d = tx; d < D; d += 16) acc = fmaf(Qs[row * D + d], Elem<TIn>::load(Kd + j * a.k_row + d), acc);
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
      m[r] = acc * a.scale_log2;
      l[r] = 1.f;
#pragma unroll
      for (int c = 0; c < kOC; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[r][c][e] = Elem<TIn>::load(Vd + j * a.v_row + c * 64 + tx * 4 + e);
    }
  }

  for (int kt = 0; kt < n_tiles; ++kt) {
    const int t0 = kt * kSimtBN;
    const int t_last = max_bound - 1;   // clamp: rows past max_bound are masked for every query
    __syncthreads();
    for (int x = tid; x < kSimtBN * kVecPerRow; x += kSimtThreads) {
      const int r = x / kVecPerRow, c = x % kVecPerRow;
      const int t = min(t0 + r, t_last);
      float f[kEpl];
      Elem<TIn>::unpack(ldg128(Kp + t * kp_row + c * kEpl), f);
#pragma unroll
      for (int e = 0; e < kEpl; ++e) Kt[(c * kEpl + e) * KP + r] = f[e];
      Elem<TIn>::unpack(ldg128(Vp + t * vp_row + c * kEpl), f);
#pragma unroll
      for (int e = 0; e < kEpl; ++e) Vs[r * D + c * kEpl + e] = f[e];
    }
    __syncthreads();

    float s[4][4];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) s[r][c] = 0.f;
#pragma unroll 4
    for (int d = 0; d < D; ++d) {
      const float4 kv = *reinterpret_cast<const float4 *>(&Kt[d * KP + tx * 4]);
      float qv[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) qv[r] = Qs[(ty * 4 + r) * D + d];
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        s[r][0] = fmaf(qv[r], kv.x, s[r][0]);
        s[r][1] = fmaf(qv[r], kv.y, s[r][1]);
        s[r][2] = fmaf(qv[r], kv.z, s[r][2]);
        s[r][3] = fmaf(qv[r], kv.w, s[r][3]);
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool vis = t0 + tx * 4 + c < bound[r];
        s[r][c] = vis ? s[r][c] * a.scale_log2 : -INFINITY;
        mx = fmaxf(mx, s[r][c]);
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m[r], mx);
      const float alpha = (m_new == -INFINITY) ? 1.f : exp2f(m[r] - m_new);
      float rs = 0.f;
      float p[4];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        p[c] = (s[r][c] == -INFINITY) ? 0.f : exp2f(s[r][c] - m_new);
        rs += p[c];
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, off);
      l[r] = l[r] * alpha + rs;
      m[r] = m_new;
#pragma unroll
      for (int c = 0; c < kOC; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[r][c][e] *= alpha;
      *reinterpret_cast<float4 *>(&Ps[(ty * 4 + r) * KP + tx * 4]) = make_float4(p[0], p[1], p[2], p[3]);
    }
    __syncthreads();
#pragma unroll 2
    for (int t = 0; t < kSimtBN; ++t) {
      float pv[4];
#pragma unroll
      for (int r = 0; r < 4; ++r) pv[r] = Ps[(ty * 4 + r) * KP + t];
#pragma unroll
      for (int c = 0; c < kOC; ++c) {
        const float4 vv = *reinterpret_cast<const float4 *>(&Vs[t * D + c * 64 + tx * 4]);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          o[r][c][0] = fmaf(pv[r], vv.x, o[r][c][0]);
          o[r][c][1] = fmaf(pv[r], vv.y, o[r][c][1]);
          o[r][c][2] = fmaf(pv[r], vv.z, o[r][c][2]);
          o[r][c][3] = fmaf(pv[r], vv.w, o[r][c][3]);
        }
      }
    }
  }

  TOut *Op = static_cast<TOut *>(a.O) + b * a.o_batch + i * a.o_inner;
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    if (!valid[r]) continue;
    const int j = j0 + ty * 4 + r;
    const float inv = 1.f / l[r];
    if (MODE == kPrefill && a.lse != nullptr && tx == 0) a.lse[(size_t)prob * a.n + j] = m[r] + log2f(l[r]);
#pragma unroll
    for (int c = 0; c < kOC; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        Elem<TOut>::store(Op + j * a.o_row + c * 64 + tx * 4 + e, o[r][c][e] * inv);
  }
}

template <typename TIn, typename TOut, int D, int MODE>
int launch_simt_attn(const SimtAttnArgs &a, int problems, cudaStream_t st) {
  constexpr size_t smem = simt_attn_smem_bytes<D>();
  auto kern = simt_attn_kernel<TIn, TOut, D, MODE>;
  AG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((a.n + kSimtBM - 1) / kSimtBM, problems);
  kern<<<grid, kSimtThreads, smem, st>>>(a);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace ag
