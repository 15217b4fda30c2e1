// The Attention-Gate pass (Sec. 3.3): AG(X) = G(MHA'(X), tau), Eq. 3 / Eq. 4,
// with the optional constant gamma inside the Sigmoid (Sec. 3.5).
//
//   1. projection   [Q' | K' | V'] = X [Wq_g | Wk_g | Wv_g]   (tcgen05 GEMM for bf16, else CUDA cores)
//   2. MHA'         H'_g = Softmax(Q'_g K'_g^T / sqrt(d'_k)) V'_g  (tcgen05 on bf16 hi/lo pairs for
//                   bf16 layers with d'_k = 128, else float32 on CUDA cores)
//   3. output layer    s = [H'_1 .. H'_h'] Wo_g;  flag = s + gamma > logit(tau)
//                   (gate_out_kernel; on the tensor-core path fused into the merge of MHA's split-K partials)
//
// The scores decide a hard threshold, so everything after the (exact) products
// of the input elements is kept in float32: a flag can then differ from an
// infinitely precise evaluation only for scores within ~1e-5 of the threshold.
#include <math.h>

#include "ag_common.cuh"
#include "attn_simt.cuh"

namespace ag {

constexpr int kGemmBM = 64, kGemmBN = 64, kGemmBK = 16;

// C[M, 3*GD] (float32) = A[M, Kd] * [W0 | W1 | W2], each W [Kd, GD] row-major.
template <typename T>
__global__ void __launch_bounds__(256)
gate_proj_kernel(const T *__restrict__ A, const T *__restrict__ W0, const T *__restrict__ W1,
                 const T *__restrict__ W2, float *__restrict__ C, int M, int Kd, int GD) {
  __shared__ __align__(16) float As[kGemmBK][kGemmBM + 4];
  __shared__ __align__(16) float Ws[kGemmBK][kGemmBN];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * kGemmBM;
  const int n0 = blockIdx.x * kGemmBN;           // column in the packed [3*GD] output
  const int which = n0 / GD, nw = n0 % GD;       // GD is a multiple of 64: a tile never straddles
  const T *W = which == 0 ? W0 : (which == 1 ? W1 : W2);
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < Kd; k0 += kGemmBK) {
    {
      const int r = tid >> 2, kq = (tid & 3) * 4;
      const int row = min(m0 + r, M - 1);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int k = k0 + kq + e;
        As[kq + e][r] = k < Kd ? Elem<T>::load(A + (size_t)row * Kd + k) : 0.f;
      }
      const int kr = tid >> 4, c4 = (tid & 15) * 4;
      const int k = k0 + kr;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        Ws[kr][c4 + e] = k < Kd ? Elem<T>::load(W + (size_t)k * GD + nw + c4 + e) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kGemmBK; ++k) {
      const float4 a = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
      const float4 w = *reinterpret_cast<const float4 *>(&Ws[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int row = m0 + ty * 4 + i;
    if (row < M)
      *reinterpret_cast<float4 *>(C + (size_t)row * 3 * GD + n0 + tx * 4) =
          make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
  }
}

// s = [H'_1 .. H'_h'] Wo_g and the threshold of Eq. 4.  One CTA = 16 tokens, one
// warp = 4 of them, lane = head (in rounds of 32 heads).  The 16 rows of H and a
// [GD][32] slice of Wo are staged in shared memory: per step of the reduction a
// warp reads one conflict-free row of Wo and four broadcast values of H.
constexpr int kOutTokens = 16, kOutThreads = 128;
template <typename T>
__global__ void __launch_bounds__(kOutThreads)
gate_out_kernel(const float *__restrict__ H, const T *__restrict__ Wo,
                const float *__restrict__ gamma, float logit_tau, int B, int n, int GD, int h,
                const int32_t *__restrict__ seq_lens, float *__restrict__ scores, uint8_t *__restrict__ flags) {
  extern __shared__ __align__(16) unsigned char sh_raw[];
  float *Hs = reinterpret_cast<float *>(sh_raw);                       // [16][GD]
  T *Ws = reinterpret_cast<T *>(sh_raw + sizeof(float) * kOutTokens * GD);   // [GD][32]
  const int tiles_per_seq = (n + kOutTokens - 1) / kOutTokens;
  const int b = blockIdx.x / tiles_per_seq, t0 = (blockIdx.x % tiles_per_seq) * kOutTokens;
  const int nt = min(kOutTokens, n - t0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float *Hg = H + ((size_t)b * n + t0) * GD;                     // rows are contiguous
  for (int x = threadIdx.x; x < kOutTokens * GD; x += kOutThreads) Hs[x] = x < nt * GD ? Hg[x] : 0.f;
  for (int i0 = 0; i0 < h; i0 += 32) {
    __syncthreads();
    for (int x = threadIdx.x; x < GD * 32; x += kOutThreads) {
      const int c = x >> 5, i = i0 + (x & 31);
      Ws[x] = i < h ? Wo[(size_t)c * h + i] : T(0.f);
    }
    __syncthreads();
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const float *hr = Hs + warp * 4 * GD;
#pragma unroll 8
    for (int c = 0; c < GD; ++c) {
      const float w = Elem<T>::load(Ws + c * 32 + lane);
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[q] = fmaf(hr[q * GD + c], w, acc[q]);
    }
    const int i = i0 + lane;
    if (i < h) {
      const float gm = gamma ? gamma[i] : 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int tt = warp * 4 + q;
        if (tt < nt) {
          const size_t o = ((size_t)b * h + i) * n + t0 + tt;
          const bool padding = seq_lens && t0 + tt >= seq_lens[b];
          if (scores) scores[o] = acc[q];
          flags[o] = !padding && (acc[q] + gm) > logit_tau ? 1 : 0;
        }
      }
    }
  }
}

size_t gate_workspace_bytes(const ag_layer_desc &d) {
  const size_t rows = (size_t)d.batch * d.seq, GD = (size_t)d.gate_heads * d.gate_head_dim;
  // [Q' | K' | V'] (float32, or the bf16 hi and lo halves), then H' (CUDA-core path) or the split-K
  // partials of MHA' (tensor-core path, where H' stays on chip)
  const size_t qkv = align_up(rows * 3 * GD * sizeof(float), 256);
  if (d.dtype == AG_BF16 && gate_attn_tc_supported(d)) return qkv + gate_attn_partial_bytes(d);
  return qkv + align_up(rows * GD * sizeof(float), 256);
}

template <typename T>
static int run_gate(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk,
                    const void *Wv, const void *Wo, const float *gamma, float *scores,
                    uint8_t *flags, void *ws, cudaStream_t st) {
  const int M = d.batch * d.seq, GD = d.gate_heads * d.gate_head_dim, Dg = d.gate_head_dim;
  float *qkv = static_cast<float *>(ws);
  float *hcat = reinterpret_cast<float *>(static_cast<char *>(ws) +
                                          align_up((size_t)M * 3 * GD * sizeof(float), 256));
  const float logit_tau = (float)log((double)d.tau / (1.0 - (double)d.tau));
  if (sizeof(T) == 2 && gate_attn_tc_supported(d)) {
    // tensor-core path: projections as bf16 hi/lo pairs, MHA' on tcgen05 with three products per term
    void *hi = ws;
    void *lo = static_cast<char *>(ws) + (size_t)M * 3 * GD * sizeof(__nv_bfloat16);
    int rc = launch_gate_proj_tc(X, Wq, Wk, Wv, nullptr, hi, lo, M, d.hidden, GD, st);
    if (rc) return rc;
    void *partials = hcat;                           // H' stays on chip: the partials take its place
    // the merge of the split-K partials carries the output layer and the threshold with it
    return launch_gate_attn_tc(d, hi, lo, partials, Wo, gamma, logit_tau, scores, flags, st);
  } else {
    if (sizeof(T) == 2 && gate_proj_tc_supported(d.hidden, GD)) {
      int rc = launch_gate_proj_tc(X, Wq, Wk, Wv, qkv, nullptr, nullptr, M, d.hidden, GD, st);
      if (rc) return rc;
    } else {
      dim3 grid(3 * GD / kGemmBN, (M + kGemmBM - 1) / kGemmBM);
      gate_proj_kernel<T><<<grid, 256, 0, st>>>(static_cast<const T *>(X), static_cast<const T *>(Wq),
                                                static_cast<const T *>(Wk), static_cast<const T *>(Wv),
                                                qkv, M, d.hidden, GD);
      AG_LAUNCH_CHECK();
    }
    SimtAttnArgs a{};
    a.Q = qkv; a.K = qkv + GD; a.V = qkv + 2 * GD; a.O = hcat;
    a.n = d.seq; a.inner = d.gate_heads;
    a.q_batch = a.k_batch = a.v_batch = (long long)d.seq * 3 * GD;
    a.q_inner = a.k_inner = a.v_inner = Dg;
    a.q_row = a.k_row = a.v_row = 3 * GD;
    a.o_batch = (long long)d.seq * GD; a.o_inner = Dg; a.o_row = GD;
    a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)Dg));
    a.seq_lens = d.seq_lens;
    const int problems = d.batch * d.gate_heads;
    int rc;
    if (Dg == 64)
      rc = d.gate_causal ? launch_simt_attn<float, float, 64, kGateCausal>(a, problems, st)
                         : launch_simt_attn<float, float, 64, kGateFull>(a, problems, st);
    else
      rc = d.gate_causal ? launch_simt_attn<float, float, 128, kGateCausal>(a, problems, st)
                         : launch_simt_attn<float, float, 128, kGateFull>(a, problems, st);
    if (rc) return rc;
  }

  const size_t out_smem = sizeof(float) * (size_t)kOutTokens * GD + sizeof(T) * (size_t)GD * 32;
  auto out_kern = gate_out_kernel<T>;
  AG_CUDA_TRY(cudaFuncSetAttribute(out_kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)out_smem));
  const int blocks = d.batch * ((d.seq + kOutTokens - 1) / kOutTokens);
  out_kern<<<blocks, kOutThreads, out_smem, st>>>(hcat, static_cast<const T *>(Wo), gamma, logit_tau,
                                                 d.batch, d.seq, GD, kv_heads_of(d), d.seq_lens, scores, flags);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int launch_gate(const ag_layer_desc &d, const void *X, const void *Wq, const void *Wk,
                const void *Wv, const void *Wo, const float *gamma, float *scores,
                uint8_t *flags, void *ws, cudaStream_t st) {
  if (d.dtype == AG_F32) return run_gate<float>(d, X, Wq, Wk, Wv, Wo, gamma, scores, flags, ws, st);
  return run_gate<__nv_bfloat16>(d, X, Wq, Wk, Wv, Wo, gamma, scores, flags, ws, st);
}

}  // namespace ag
