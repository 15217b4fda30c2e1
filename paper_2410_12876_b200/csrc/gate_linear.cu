// The local gate of Sec. 3.4 ("Local or global?", ablation setting (5)): MHA' is
// replaced by one linear layer, s = X W_lin, followed by the threshold of Eq. 4
// (gamma of Sec. 3.5 inside the Sigmoid).  A token's flag depends on its own
// hidden state only.
//
// s is a skinny contraction, [B n, d] x [d, h] with h a few dozen columns: the
// kernel is bound by reading X once.  bf16 layers run on the tensor cores
// (products of bf16 inputs are exact in the float32 accumulator): one CTA owns
// 128 tokens and a slice of d; the CTAs of a thread-block cluster split d among
// them so that enough CTAs stream X, and the cluster's first CTA adds the
// partial accumulators in rank order through distributed shared memory (a fixed
// order: results do not vary from run to run), thresholds and writes.
//   A = X      [B n, d]  row-major -> K-major operand, 128-byte swizzled rows
//   B = W_lin  [d, h]    row-major -> MN-major operand: one panel of [64 k][64 n],
//                                     columns past h filled with zeros by TMA
// Other layers (float32, h > 64, odd strides) take a CUDA-core kernel.
#include <cooperative_groups.h>
#include <math.h>

#include "ag_common.cuh"
#include "umma.cuh"

namespace ag {

using namespace umma;
namespace cg = cooperative_groups;

constexpr int kGlBM = 128, kGlBK = 64, kGlThreads = 192, kGlStages = 6;
constexpr int kGlABytes = kGlBM * kGlBK * 2;              // 16 KB
constexpr int kGlBBytes = kGlBK * 64 * 2;                 // one panel [64 k][64 n] = 8 KB
constexpr int kGlStageBytes = kGlABytes + kGlBBytes;
constexpr int kGlMaxN = 64;                               // heads the tensor-core kernel serves
constexpr int kGlPartBytes = kGlBM * kGlMaxN * 4;         // a CTA's partial accumulator, [col][row]
constexpr int kGlSmemBytes = kGlStages * kGlStageBytes + kGlPartBytes + 1024 /*align*/ + 256 /*barriers*/;
constexpr uint32_t kGlTmemCols = 64;

struct GateLinearArgs {
  const int32_t *seq_lens;   // [B] or NULL: tokens past seq_lens[b] are padding (flag 0)
  const float *gamma;
  float *scores;
  uint8_t *flags;
  int M, n, h, kb_total, kb_per_cta;   // tokens, sequence length, heads, 64-wide k blocks in all / per CTA
  float logit_tau;
};

template <int N>   // MMA width: heads rounded up to 32
__global__ void __launch_bounds__(kGlThreads, 1)
gate_linear_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
                      const GateLinearArgs a) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float *part = reinterpret_cast<float *>(smem + kGlStages * kGlStageBytes);          // [N][128]
  uint64_t *full = reinterpret_cast<uint64_t *>(smem + kGlStages * kGlStageBytes + kGlPartBytes);
  uint64_t *empty = full + kGlStages;
  uint64_t *acc_full = empty + kGlStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);

  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank(), nranks = (int)cluster.num_blocks();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * kGlBM;
  const int kb_begin = rank * a.kb_per_cta;
  const int num_kb = max(0, min(a.kb_total, kb_begin + a.kb_per_cta) - kb_begin);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kGlStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    fence_barrier_init();
    prefetch_tensormap(&tmX);
    prefetch_tensormap(&tmW);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kGlTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_acc = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kGlStages;
        const uint32_t ph = (kb / kGlStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1)) break;
        uint8_t *sa = smem + s * kGlStageBytes, *sb = sa + kGlABytes;
        mbar_arrive_expect_tx(&full[s], kGlStageBytes);
        tma_load_2d(sa, &tmX, &full[s], (kb_begin + kb) * kGlBK, m0);
        tma_load_2d(sb, &tmW, &full[s], 0, (kb_begin + kb) * kGlBK);
      }
    }
  } else if (warp == 1) {
    // every lane runs the control flow (operands stay warp-uniform); one elected lane issues
    constexpr uint32_t idesc = idesc_bf16_f32(kGlBM, N, false, true);
    const uint64_t da0 = desc_kmajor_sw128(smem_u32(smem));
    const uint64_t db0 = desc_mnmajor_sw128(smem_u32(smem) + kGlABytes, kGlBBytes);
    const uint32_t a_lo0 = (uint32_t)da0, a_hi = (uint32_t)(da0 >> 32);
    const uint32_t b_lo0 = (uint32_t)db0, b_hi = (uint32_t)(db0 >> 32);
    bool ok = true;
    for (int kb = 0; kb < num_kb && ok; ++kb) {
      const int s = kb % kGlStages;
      const uint32_t ph = (kb / kGlStages) & 1;
      ok = mbar_wait(&full[s], ph);
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t a_lo = a_lo0 + ((s * kGlStageBytes) >> 4), b_lo = b_lo0 + ((s * kGlStageBytes) >> 4);
      if (elect_one()) {
#pragma unroll
        for (int k = 0; k < kGlBK / 16; ++k)
          mma_ss_lohi(tmem_acc, a_lo + ((k * 32) >> 4), a_hi, b_lo + ((k * 2048) >> 4), b_hi, idesc, (kb | k) != 0);
        mma_commit(&empty[s]);
      }
      __syncwarp();
    }
    if (elect_one()) mma_commit(acc_full);   // accumulator complete (or unwinding)
    __syncwarp();
  } else {
    // this CTA's partial sums: thread = token row, into shared memory as [col][row]
    const int quad = warp & 3, r_in = quad * 32 + lane;
    const bool ok = mbar_wait(acc_full, 0);
    tc_fence_after_sync();
#pragma unroll
    for (int c = 0; c < N; c += 32) {
      uint32_t r[32];
      if (ok && num_kb > 0) {
        tmem_ld_x32_sync(tmem_acc + ((uint32_t)(quad * 32) << 16) + c, r);
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) r[e] = 0u;
      }
#pragma unroll
      for (int e = 0; e < 32; ++e) part[(c + e) * kGlBM + r_in] = __uint_as_float(r[e]);
    }
  }
  cluster.sync();                       // every CTA's partial sums are in its shared memory
  if (rank == 0 && warp >= 2) {
    const int quad = warp & 3, r_in = quad * 32 + lane;
    const int tok = m0 + r_in;
    if (tok < a.M) {
      const int b = tok / a.n, t = tok % a.n;
      const bool padding = a.seq_lens && t >= a.seq_lens[b];
      float s[N];
#pragma unroll
      for (int i = 0; i < N; ++i) s[i] = 0.f;
      for (int rk = 0; rk < nranks; ++rk) {          // rank order: the sum does not depend on timing
        const float *p = cluster.map_shared_rank(part, rk) + r_in;
#pragma unroll
        for (int i = 0; i < N; ++i) s[i] += p[i * kGlBM];   // independent loads, all in flight
      }
#pragma unroll
      for (int i = 0; i < N; ++i) {
        if (i < a.h) {
          const size_t o = ((size_t)b * a.h + i) * a.n + t;   // lanes = consecutive tokens: coalesced
          if (a.scores) a.scores[o] = s[i];
          a.flags[o] = !padding && (s[i] + (a.gamma ? a.gamma[i] : 0.f)) > a.logit_tau ? 1 : 0;
        }
      }
    }
  }
  cluster.sync();                       // partial sums stay alive until the first CTA has read them
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_acc, kGlTmemCols);
}

// CUDA-core form: one warp per token, lanes stride over d, heads in registers eight at a time.
template <typename T>
__global__ void __launch_bounds__(256)
gate_linear_simt_kernel(const T *__restrict__ X, const T *__restrict__ W, const float *__restrict__ gamma,
                        float logit_tau, int M, int n, int d, int h, const int32_t *__restrict__ seq_lens,
                        float *__restrict__ scores, uint8_t *__restrict__ flags) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tok = blockIdx.x * 8 + warp;
  if (tok >= M) return;
  const int b = tok / n, t = tok % n;
  const T *x = X + (size_t)tok * d;
  for (int i0 = 0; i0 < h; i0 += 8) {
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int k = lane; k < d; k += 32) {
      const float xv = Elem<T>::load(x + k);
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (i0 + e < h) acc[e] = fmaf(xv, Elem<T>::load(W + (size_t)k * h + i0 + e), acc[e]);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], off);
    }
    if (lane == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int i = i0 + e;
        if (i < h) {
          const size_t o = ((size_t)b * h + i) * n + t;
          if (scores) scores[o] = acc[e];
          flags[o] = !(seq_lens && t >= seq_lens[b]) && (acc[e] + (gamma ? gamma[i] : 0.f)) > logit_tau ? 1 : 0;
        }
      }
    }
  }
}

template <int N>
static int run_gate_linear_tc(const ag_layer_desc &d, const void *X, const void *W, const GateLinearArgs &a0,
                              cudaStream_t st) {
  GateLinearArgs a = a0;
  CUtensorMap tmX, tmW;
  int rc = make_tmap_2d_bf16(&tmX, X, a.M, d.hidden, (uint64_t)d.hidden * 2, kGlBM, kGlBK);
  if (rc) return rc;
  rc = make_tmap_2d_bf16(&tmW, W, d.hidden, kv_heads_of(d), (uint64_t)kv_heads_of(d) * 2, kGlBK, 64);
  if (rc) return rc;
  // split d over a cluster until about one CTA per SM streams X (at least four k blocks each)
  const int m_tiles = (a.M + kGlBM - 1) / kGlBM;
  int split = 1;
  while (split < 8 && m_tiles * split * 2 <= 160 && a.kb_total / (split * 2) >= 4) split *= 2;
  a.kb_per_cta = (a.kb_total + split - 1) / split;
  auto kern = gate_linear_tc_kernel<N>;
  AG_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kGlSmemBytes));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(split, m_tiles);
  cfg.blockDim = dim3(kGlThreads);
  cfg.dynamicSmemBytes = kGlSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = split; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmX, tmW, a));
  return AG_OK;
}

int launch_gate_linear(const ag_layer_desc &d, const void *X, const void *W, const float *gamma,
                       float *scores, uint8_t *flags, cudaStream_t st) {
  GateLinearArgs a;
  a.seq_lens = d.seq_lens; a.gamma = gamma; a.scores = scores; a.flags = flags;
  a.M = d.batch * d.seq; a.n = d.seq; a.h = kv_heads_of(d);
  a.kb_total = (d.hidden + kGlBK - 1) / kGlBK; a.kb_per_cta = a.kb_total;
  a.logit_tau = (float)log((double)d.tau / (1.0 - (double)d.tau));
  const bool tc = d.dtype == AG_BF16 && kv_heads_of(d) <= kGlMaxN && kv_heads_of(d) % 8 == 0 && d.hidden % 8 == 0 &&
                  (int64_t)d.batch * d.seq < ((int64_t)1 << 31) - kGlBM && (a.M + kGlBM - 1) / kGlBM <= 65535;
  if (tc) {
    if (kv_heads_of(d) <= 32) return run_gate_linear_tc<32>(d, X, W, a, st);
    return run_gate_linear_tc<64>(d, X, W, a, st);
  }
  const int blocks = (a.M + 7) / 8;
  if (d.dtype == AG_F32)
    gate_linear_simt_kernel<float><<<blocks, 256, 0, st>>>(static_cast<const float *>(X), static_cast<const float *>(W),
                                                          gamma, a.logit_tau, a.M, a.n, d.hidden, kv_heads_of(d), d.seq_lens, scores, flags);
  else
    gate_linear_simt_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(
        static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(W), gamma, a.logit_tau, a.M, a.n,
        d.hidden, kv_heads_of(d), d.seq_lens, scores, flags);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int gate_linear_wait_timeouts() {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, umma::g_wait_expired, sizeof(int)) != cudaSuccess) return -1;
  return v;
}

}  // namespace ag
