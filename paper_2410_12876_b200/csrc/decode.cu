// Single-query decode attention over the ragged retained cache (Sec. 3.1
// decoding stage; cache = retained tokens only, Sec. 3.3; the new token always
// sees its own key, Eq. 5 case j = t).
//
// Split-K: slab s = (sequence, head) is cut into chunks of rows; a chunk is
// reduced to an un-normalised (o, m, l) triple, and the chunks of a slab are
// merged with the self term (q . k_new, v_new) and normalised.  The work is
// HBM-bound: every cache row is read exactly once with 16-byte vector loads,
// one row per group of kLanes consecutive lanes, several rows in flight per lane.
//
// Two forms.  Few slabs (a launch is latency-bound): one thread-block cluster
// per slab, one chunk per CTA, the triples merged through distributed shared
// memory by the cluster's first CTA - one kernel, no scratch.  Many slabs:
// decode_partial_kernel writes the triples of up to kMaxSplits chunks per slab
// to the workspace and decode_combine_kernel merges them.
#include <cooperative_groups.h>
#include <math.h>
#include <nvtx3/nvToolsExt.h>

#include <type_traits>

#include "ag_common.cuh"
#include "decode_mma_core.cuh"

namespace ag {

constexpr int kMaxSplits = 32;     // chunks per slab the workspace is sized for
constexpr int kPartThreads = 256;
constexpr int kUnroll = 8;         // rows in flight per lane group (x2: K and V)
constexpr int kClusterMaxSlabs = 64;    // up to here one cluster per slab; beyond, split-K through the workspace
constexpr int kClusterThreads = 512;    // 256 rows in flight per CTA of a cluster (bf16, D = 128)

// Grouped-query attention: slab s = (sequence, query head) of q and o reads the cache slab, k_new
// and v_new of its key/value head.
struct HeadMap {
  int heads, kv_heads;
  __device__ __forceinline__ int kv_slab(int slab) const {
    return (slab / heads) * kv_heads + (slab % heads) / (heads / kv_heads);
  }
};

// The conditional append of the decoding stage (Sec. 3.1 with the gate's flag for the new token),
// for kernels that carry it with the attention of the same step: flag_new = NULL means no append.
struct AppendArgs {
  const uint8_t *flag_new;   // [slabs] or NULL
  const int32_t *cap;
  int32_t *len;
  void *k_rows, *v_rows;
  int32_t *dev_status;
};
// Called by the threads [first, first + row vectors) of ONE CTA per slab (every thread may call, the
// others return), after every read of len[slab] and of the slab's rows by this launch has
// completed.  L = the length those reads saw.
template <typename T, int D>
__device__ __forceinline__ void append_new_row(const AppendArgs &ap, int slab, int L, int64_t row0,
                                               const T *__restrict__ k_new, const T *__restrict__ v_new,
                                               int first = 0) {
  constexpr int kVecs = D * (int)sizeof(T) / 16;
  const int vec = (int)threadIdx.x - first;
  if (ap.flag_new == nullptr || vec < 0 || vec >= kVecs || ap.flag_new[slab] == 0) return;
  if (L >= ap.cap[slab]) {
    if (vec == 0 && ap.dev_status) atomicOr(ap.dev_status, AG_DEV_OVERFLOW);
    return;
  }
  const size_t dst = ((size_t)row0 + L) * D * sizeof(T) + vec * 16;
  const size_t src = (size_t)slab * D * sizeof(T) + vec * 16;
  *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(ap.k_rows) + dst) =
      *reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(k_new) + src);
  *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(ap.v_rows) + dst) =
      *reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(v_new) + src);
  if (vec == 0) ap.len[slab] = L + 1;
}

// Recent-token window: scores of the query against the ring of its key/value slab, by every warp
// of the CTA: sm_s[r] = scale_log2 * q . k_r for a live slot (an evicted token the query still
// sees), -inf otherwise.  The caller synchronises the CTA before reading sm_s.
template <typename T, int D>
__device__ __forceinline__ void ring_scores(const RecentRing &rg, int kv, const T *__restrict__ q_row,
                                            float scale_log2, float *sm_s) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int r = warp; r < rg.R; r += n_warps) {
    const T *kr = static_cast<const T *>(rg.k) + ((size_t)kv * rg.R + r) * D;
    float a = 0.f;
#pragma unroll
    for (int d = lane; d < D; d += 32) a = fmaf(Elem<T>::load(q_row + d), Elem<T>::load(kr + d), a);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
    if (lane == 0) sm_s[r] = rg.live[(size_t)kv * rg.R + r] != 0 ? a * scale_log2 : -INFINITY;
  }
}

// Rows [r_begin, r_end) of one slab, streamed by a whole CTA of kThreads threads: thread (g, v) =
// (row group, 16-byte slice of the row) ends with its group's running maximum m, sum l and slice
// of o (log2 domain).
template <typename T, int D, int kThreads>
__device__ __forceinline__ void decode_stream_rows(const T *__restrict__ q, const T *__restrict__ k_rows,
                                                   const T *__restrict__ v_rows, int64_t row0, int slab,
                                                   int r_begin, int r_end, float scale_log2, float &m,
                                                   float &l, float (&o)[Elem<T>::kPerVec]) {
  constexpr int kEpl = Elem<T>::kPerVec;        // elements per lane
  constexpr int kLanes = D / kEpl;              // lanes per row
  constexpr int kGroups = kThreads / kLanes;
  const int g = threadIdx.x / kLanes, v = threadIdx.x % kLanes;

  float qf[kEpl];
  Elem<T>::unpack(ldg128(q + (size_t)slab * D + v * kEpl), qf);
#pragma unroll
  for (int e = 0; e < kEpl; ++e) qf[e] *= scale_log2;

  const T *Kb = k_rows + (size_t)row0 * D + v * kEpl;
  const T *Vb = v_rows + (size_t)row0 * D + v * kEpl;

  m = -INFINITY; l = 0.f;
#pragma unroll
  for (int e = 0; e < kEpl; ++e) o[e] = 0.f;

  // The trip count is the same for every thread of the CTA (the shuffles below
  // need whole warps); rows past r_end are clamped for the load and get weight 0.
  for (int r0 = r_begin; r0 < r_end; r0 += kUnroll * kGroups) {
    const int r = r0 + g;
    uint4 kv[kUnroll], vv[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int ru = min(r + u * kGroups, r_end - 1);
      kv[u] = ldg128_stream(Kb + (size_t)ru * D);
      vv[u] = ldg128_stream(Vb + (size_t)ru * D);
    }
    float s[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float kf[kEpl];
      Elem<T>::unpack(kv[u], kf);
      float a = 0.f;
#pragma unroll
      for (int e = 0; e < kEpl; ++e) a = fmaf(qf[e], kf[e], a);
#pragma unroll
      for (int off = kLanes / 2; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
      s[u] = (r + u * kGroups < r_end) ? a : -INFINITY;
    }
    float m_new = m;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) m_new = fmaxf(m_new, s[u]);
    // a group may not have seen a valid row yet: keep everything at zero then
    const float alpha = (m_new == -INFINITY) ? 1.f : exp2f(m - m_new);
    l *= alpha;
#pragma unroll
    for (int e = 0; e < kEpl; ++e) o[e] *= alpha;
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const float p = (s[u] == -INFINITY) ? 0.f : exp2f(s[u] - m_new);
      l += p;
      float vf[kEpl];
      Elem<T>::unpack(vv[u], vf);
#pragma unroll
      for (int e = 0; e < kEpl; ++e) o[e] = fmaf(p, vf[e], o[e]);
    }
    m = m_new;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kPartThreads)
decode_partial_kernel(const T *__restrict__ q, const T *__restrict__ k_rows,
                      const T *__restrict__ v_rows, const int64_t *__restrict__ row_off,
                      const int32_t *__restrict__ len, float scale_log2, int chunk_rows,
                      float *__restrict__ part_o, float *__restrict__ part_ml, const HeadMap hm) {
  constexpr int kEpl = Elem<T>::kPerVec;
  constexpr int kLanes = D / kEpl;
  constexpr int kGroups = kPartThreads / kLanes;
  const int slab = blockIdx.y, chunk = blockIdx.x;
  const int kv = hm.kv_slab(slab);
  const int L = len[kv];
  const int r_begin = chunk * chunk_rows;
  if (r_begin >= L) return;
  const int r_end = min(L, r_begin + chunk_rows);
  const int g = threadIdx.x / kLanes, v = threadIdx.x % kLanes;
  float m, l, o[kEpl];
  decode_stream_rows<T, D, kPartThreads>(q, k_rows, v_rows, row_off[kv], slab, r_begin, r_end, scale_log2, m, l, o);

  __shared__ float sm_m[kGroups], sm_l[kGroups];
  __shared__ float sm_o[kGroups][D];
  if (v == 0) { sm_m[g] = m; sm_l[g] = l; }
#pragma unroll
  for (int e = 0; e < kEpl; ++e) sm_o[g][v * kEpl + e] = o[e];
  __syncthreads();
  float mc = -INFINITY;
#pragma unroll
  for (int i = 0; i < kGroups; ++i) mc = fmaxf(mc, sm_m[i]);
  float *po = part_o + ((size_t)slab * kMaxSplits + chunk) * D;
  for (int d = threadIdx.x; d < D; d += kPartThreads) {
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kGroups; ++i) acc = fmaf(sm_m[i] == -INFINITY ? 0.f : exp2f(sm_m[i] - mc), sm_o[i][d], acc);
    po[d] = acc;
  }
  if (threadIdx.x == 0) {
    float lc = 0.f;
#pragma unroll
    for (int i = 0; i < kGroups; ++i) lc = fmaf(sm_m[i] == -INFINITY ? 0.f : exp2f(sm_m[i] - mc), sm_l[i], lc);
    part_ml[((size_t)slab * kMaxSplits + chunk) * 2 + 0] = mc;
    part_ml[((size_t)slab * kMaxSplits + chunk) * 2 + 1] = lc;
  }
}

// Grouped-query form of the chunk pass: one CTA streams a chunk of a KEY/VALUE slab once for the
// G query heads that share it (G = 2 or 4; rows in flight per lane group halved to make room for
// G running softmaxes per thread) and leaves one triple per query head, where
// decode_combine_kernel expects it.
constexpr int kUnrollGqa = 4;
template <typename T, int D, int G>
__global__ void __launch_bounds__(kPartThreads)
decode_partial_gqa_kernel(const T *__restrict__ q, const T *__restrict__ k_rows,
                          const T *__restrict__ v_rows, const int64_t *__restrict__ row_off,
                          const int32_t *__restrict__ len, float scale_log2, int chunk_rows,
                          float *__restrict__ part_o, float *__restrict__ part_ml, int kv_heads) {
  constexpr int kEpl = Elem<T>::kPerVec;
  constexpr int kLanes = D / kEpl;
  constexpr int kGroups = kPartThreads / kLanes;
  const int kv = blockIdx.y, chunk = blockIdx.x;
  const int slab0 = (kv / kv_heads) * kv_heads * G + (kv % kv_heads) * G;   // first query slab of the group
  const int L = len[kv];
  const int r_begin = chunk * chunk_rows;
  if (r_begin >= L) return;
  const int r_end = min(L, r_begin + chunk_rows);
  const int g = threadIdx.x / kLanes, v = threadIdx.x % kLanes;

  float qf[G][kEpl], o[G][kEpl], m[G], l[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    Elem<T>::unpack(ldg128(q + (size_t)(slab0 + h) * D + v * kEpl), qf[h]);
    m[h] = -INFINITY; l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < kEpl; ++e) { qf[h][e] *= scale_log2; o[h][e] = 0.f; }
  }
  const T *Kb = k_rows + (size_t)row_off[kv] * D + v * kEpl;
  const T *Vb = v_rows + (size_t)row_off[kv] * D + v * kEpl;

  // uniform trip count (the shuffles need whole warps); rows past r_end are clamped and get weight 0
  for (int r0 = r_begin; r0 < r_end; r0 += kUnrollGqa * kGroups) {
    const int r = r0 + g;
    uint4 kv4[kUnrollGqa], vv4[kUnrollGqa];
#pragma unroll
    for (int u = 0; u < kUnrollGqa; ++u) {
      const int ru = min(r + u * kGroups, r_end - 1);
      kv4[u] = ldg128_stream(Kb + (size_t)ru * D);
      vv4[u] = ldg128_stream(Vb + (size_t)ru * D);
    }
    float sc[kUnrollGqa][G];
#pragma unroll
    for (int u = 0; u < kUnrollGqa; ++u) {
      float kf[kEpl];
      Elem<T>::unpack(kv4[u], kf);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float a = 0.f;
#pragma unroll
        for (int e = 0; e < kEpl; ++e) a = fmaf(qf[h][e], kf[e], a);
#pragma unroll
        for (int off = kLanes / 2; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
        sc[u][h] = (r + u * kGroups < r_end) ? a : -INFINITY;
      }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      float m_new = m[h];
#pragma unroll
      for (int u = 0; u < kUnrollGqa; ++u) m_new = fmaxf(m_new, sc[u][h]);
      const float alpha = (m_new == -INFINITY) ? 1.f : exp2f(m[h] - m_new);
      l[h] *= alpha;
#pragma unroll
      for (int e = 0; e < kEpl; ++e) o[h][e] *= alpha;
#pragma unroll
      for (int u = 0; u < kUnrollGqa; ++u) {
        const float p = (sc[u][h] == -INFINITY) ? 0.f : exp2f(sc[u][h] - m_new);
        l[h] += p;
        float vf[kEpl];
        Elem<T>::unpack(vv4[u], vf);
#pragma unroll
        for (int e = 0; e < kEpl; ++e) o[h][e] = fmaf(p, vf[e], o[h][e]);
      }
      m[h] = m_new;
    }
  }

  __shared__ float sm_m[G][kGroups], sm_l[G][kGroups];
  __shared__ float sm_o[kGroups][D];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    __syncthreads();                                 // sm_o of the previous head has been read
    if (v == 0) { sm_m[h][g] = m[h]; sm_l[h][g] = l[h]; }
#pragma unroll
    for (int e = 0; e < kEpl; ++e) sm_o[g][v * kEpl + e] = o[h][e];
    __syncthreads();
    float mc = -INFINITY;
#pragma unroll
    for (int i = 0; i < kGroups; ++i) mc = fmaxf(mc, sm_m[h][i]);
    const size_t slot = (size_t)(slab0 + h) * kMaxSplits + chunk;
    for (int d = threadIdx.x; d < D; d += kPartThreads) {
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < kGroups; ++i)
        acc = fmaf(sm_m[h][i] == -INFINITY ? 0.f : exp2f(sm_m[h][i] - mc), sm_o[i][d], acc);
      part_o[slot * D + d] = acc;
    }
    if (threadIdx.x == 0) {
      float lc = 0.f;
#pragma unroll
      for (int i = 0; i < kGroups; ++i) lc = fmaf(sm_m[h][i] == -INFINITY ? 0.f : exp2f(sm_m[h][i] - mc), sm_l[h][i], lc);
      part_ml[slot * 2 + 0] = mc;
      part_ml[slot * 2 + 1] = lc;
    }
  }
}

// One CTA of D threads per slab: thread d owns output dimension d.
template <typename T, int D>
__global__ void __launch_bounds__(D)
decode_combine_kernel(const T *__restrict__ q, const T *__restrict__ k_new,
                      const T *__restrict__ v_new, const int32_t *len,
                      float scale_log2, int chunk_rows, const float *__restrict__ part_o,
                      const float *__restrict__ part_ml, T *__restrict__ o,
                      const int64_t *__restrict__ row_off, const AppendArgs ap, const HeadMap hm,
                      const RecentRing rg) {
  const int slab = blockIdx.x, d = threadIdx.x;
  const int kv = hm.kv_slab(slab);
  const int L = len[kv];
  const int n_chunks = (L + chunk_rows - 1) / chunk_rows;
  __shared__ float red[D / 32];
  __shared__ float ring_s[kMaxRecent];
  float a = Elem<T>::load(q + (size_t)slab * D + d) * Elem<T>::load(k_new + (size_t)kv * D + d);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
  if ((d & 31) == 0) red[d >> 5] = a;
  ring_scores<T, D>(rg, kv, q + (size_t)slab * D, scale_log2, ring_s);
  __syncthreads();
  // Every thread of the CTA has read the slab's length (above the barrier), and the chunk pass, the
  // only reader of the slab's rows, has completed: the new row may go in and the length may move.
  // (Never asked for when query heads share a slab: another head's CTA may still be reading its length.)
  append_new_row<T, D>(ap, kv, L, row_off[kv], k_new, v_new);
  float s_self = 0.f;
#pragma unroll
  for (int i = 0; i < D / 32; ++i) s_self += red[i];
  s_self *= scale_log2;
  const float *pml = part_ml + (size_t)slab * kMaxSplits * 2;
  float m = s_self;
  for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, pml[2 * c]);
  for (int r = 0; r < rg.R; ++r) m = fmaxf(m, ring_s[r]);
  const float w_self = exp2f(s_self - m);
  float acc = w_self * Elem<T>::load(v_new + (size_t)kv * D + d);
  float l = w_self;
  const float *po = part_o + (size_t)slab * kMaxSplits * D + d;
  for (int c = 0; c < n_chunks; ++c) {
    const float w = exp2f(pml[2 * c] - m);
    acc = fmaf(w, po[(size_t)c * D], acc);
    l = fmaf(w, pml[2 * c + 1], l);
  }
  // the evicted tokens of the recent-token window
  for (int r = 0; r < rg.R; ++r) {
    if (ring_s[r] == -INFINITY) continue;
    const float w = exp2f(ring_s[r] - m);
    acc = fmaf(w, Elem<T>::load(static_cast<const T *>(rg.v) + ((size_t)kv * rg.R + r) * D + d), acc);
    l += w;
  }
  Elem<T>::store(o + (size_t)slab * D + d, acc / l);
  if (rg.R > 0 && ap.flag_new != nullptr) {
    // the step carries the append: the new token joins the ring once every thread has read it
    constexpr int kVecs = D * (int)sizeof(T) / 16;
    __syncthreads();
    if (d < kVecs)
      ring_put<kVecs>(rg, kv, d, reinterpret_cast<const uint8_t *>(k_new + (size_t)kv * D),
                      reinterpret_cast<const uint8_t *>(v_new + (size_t)kv * D), ap.flag_new[kv] != 0);
  }
}

// One cluster of kClusterSize CTAs per slab.  CTA `rank` reduces rows [rank, rank + 1) * per of
// the slab to a triple in its own shared memory; after a cluster barrier the first CTA reads all
// triples through distributed shared memory, adds the self term and writes the output.  The
// second barrier keeps every CTA's shared memory alive until it has been read.  No CTA leaves
// early: the cluster barriers need all of them.
constexpr int kClusterSize = 8;
template <typename T, int D, int kThreads>
__global__ void __launch_bounds__(kThreads)
decode_cluster_kernel(const T *__restrict__ q, const T *__restrict__ k_new, const T *__restrict__ v_new,
                      const T *__restrict__ k_rows, const T *__restrict__ v_rows,
                      const int64_t *__restrict__ row_off, const int32_t *len,
                      float scale_log2, T *__restrict__ out, const AppendArgs ap, const HeadMap hm,
                      const RecentRing rg) {
  namespace cg = cooperative_groups;
  constexpr int kEpl = Elem<T>::kPerVec;
  constexpr int kLanes = D / kEpl;
  constexpr int kGroups = kThreads / kLanes;
  cg::cluster_group cluster = cg::this_cluster();
  const int slab = blockIdx.y, rank = (int)cluster.block_rank();
  const int kv = hm.kv_slab(slab);
  pdl_launch_dependents();
  pdl_wait();
  const int L = len[kv];
  const int per = ((L + kClusterSize - 1) / kClusterSize + kGroups - 1) / kGroups * kGroups;
  const int r_begin = min(L, rank * per), r_end = min(L, r_begin + per);
  const int g = threadIdx.x / kLanes, v = threadIdx.x % kLanes;

  __shared__ float sm_m[kGroups], sm_l[kGroups];
  __shared__ float sm_o[kGroups][D];
  __shared__ float cta_o[D];          // this CTA's triple, read by the first CTA of the cluster
  __shared__ float cta_ml[2];
  __shared__ float red[D / 32];
  __shared__ float ring_s[kMaxRecent];

  // self score q . k_new: only the first CTA needs it; its loads are in flight with the stream's
  // (and the new value, which the merge after the cluster barrier would otherwise wait for)
  float prod = 0.f, v_self = 0.f;
  if (rank == 0 && threadIdx.x < D) {
    prod = Elem<T>::load(q + (size_t)slab * D + threadIdx.x) * Elem<T>::load(k_new + (size_t)kv * D + threadIdx.x);
    v_self = Elem<T>::load(v_new + (size_t)kv * D + threadIdx.x);
  }

  float m, l, o[kEpl];
  decode_stream_rows<T, D, kThreads>(q, k_rows, v_rows, row_off[kv], slab, r_begin, r_end, scale_log2, m, l, o);

  if (v == 0) { sm_m[g] = m; sm_l[g] = l; }
#pragma unroll
  for (int e = 0; e < kEpl; ++e) sm_o[g][v * kEpl + e] = o[e];
  if (threadIdx.x < D) {              // whole warps: D is a multiple of 32
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) prod += __shfl_xor_sync(0xffffffffu, prod, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = prod;
  }
  if (rank == 0) ring_scores<T, D>(rg, kv, q + (size_t)slab * D, scale_log2, ring_s);
  __syncthreads();
  float mc = -INFINITY;
#pragma unroll
  for (int i = 0; i < kGroups; ++i) mc = fmaxf(mc, sm_m[i]);
  if (threadIdx.x < D) {
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < kGroups; ++i)
      acc = fmaf(sm_m[i] == -INFINITY ? 0.f : exp2f(sm_m[i] - mc), sm_o[i][threadIdx.x], acc);
    cta_o[threadIdx.x] = acc;
  }
  if (threadIdx.x == 0) {
    float lc = 0.f;
#pragma unroll
    for (int i = 0; i < kGroups; ++i) lc = fmaf(sm_m[i] == -INFINITY ? 0.f : exp2f(sm_m[i] - mc), sm_l[i], lc);
    cta_ml[0] = mc;
    cta_ml[1] = lc;
  }
  cluster.sync();
  // every CTA of the cluster has read the length and its rows: the new row may go in
  // (never asked for when query heads share a slab: another head's cluster may still be reading its length)
  // by threads that have no part in the merge below, so that the two run side by side
  if (rank == 0) append_new_row<T, D>(ap, kv, L, row_off[kv], k_new, v_new, D);
  if (rank == 0 && threadIdx.x < D) {
    const int d = threadIdx.x;
    float s_self = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) s_self += red[i];
    s_self *= scale_log2;
    float mr[kClusterSize], lr[kClusterSize], orr[kClusterSize];
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) {
      const float *ml = cluster.map_shared_rank(cta_ml, r);
      mr[r] = ml[0];
      lr[r] = ml[1];
      orr[r] = cluster.map_shared_rank(cta_o, r)[d];
    }
    float mm = s_self;
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) mm = fmaxf(mm, mr[r]);
    for (int r = 0; r < rg.R; ++r) mm = fmaxf(mm, ring_s[r]);
    const float w_self = exp2f(s_self - mm);
    float acc = w_self * v_self;
    float lsum = w_self;
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) {
      const float w = mr[r] == -INFINITY ? 0.f : exp2f(mr[r] - mm);
      acc = fmaf(w, orr[r], acc);
      lsum = fmaf(w, lr[r], lsum);
    }
    // the evicted tokens of the recent-token window
    for (int r = 0; r < rg.R; ++r) {
      if (ring_s[r] == -INFINITY) continue;
      const float w = exp2f(ring_s[r] - mm);
      acc = fmaf(w, Elem<T>::load(static_cast<const T *>(rg.v) + ((size_t)kv * rg.R + r) * D + d), acc);
      lsum += w;
    }
    Elem<T>::store(out + (size_t)slab * D + d, acc / lsum);
  }
  if (rank == 0 && rg.R > 0 && ap.flag_new != nullptr) {
    // the step carries the append: the new token joins the ring once every thread has read it
    constexpr int kVecs = D * (int)sizeof(T) / 16;
    __syncthreads();
    if ((int)threadIdx.x < kVecs)
      ring_put<kVecs>(rg, kv, threadIdx.x, reinterpret_cast<const uint8_t *>(k_new + (size_t)kv * D),
                      reinterpret_cast<const uint8_t *>(v_new + (size_t)kv * D), ap.flag_new[kv] != 0);
  }
  cluster.sync();
}

// The cluster form for bf16, head_dim 128, with the rows streamed through shared memory and the
// scores and weighted sums on warp-level MMAs (decode_mma_core.cuh; the query is row 0 of the 16-row
// operand): per row a fraction of the instructions of the CUDA-core form, which at these sizes is
// bound by instruction issue and by what one SM can take in, not by latency alone.  CTA `rank`
// takes whole 64-row tiles; everything after the streaming is as in decode_cluster_kernel.
// three stages: a CTA has few tiles and no neighbour to hide behind, so two of them are kept in flight
constexpr int kCmStages = 3;
__global__ void __launch_bounds__(kGqThreads, 2)
decode_cluster_mma_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_new,
                          const __nv_bfloat16 *__restrict__ v_new, const __nv_bfloat16 *__restrict__ k_rows,
                          const __nv_bfloat16 *__restrict__ v_rows, const int64_t *__restrict__ row_off,
                          const int32_t *len, float scale_log2, __nv_bfloat16 *__restrict__ out,
                          const AppendArgs ap, const HeadMap hm, const RecentRing rg) {
  namespace cg = cooperative_groups;
  using T = __nv_bfloat16;
  constexpr int D = kGqD;
  static_assert(kGqThreads == D, "one thread per output dimension in the merge");
  extern __shared__ __align__(128) uint8_t gq_smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int slab = blockIdx.y, rank = (int)cluster.block_rank();
  const int kv = hm.kv_slab(slab);
  const int d = threadIdx.x;
  pdl_launch_dependents();
  // the slab's first row never changes once the cache is laid out: read ahead of the wait for the
  // preceding kernel, so that only the length is on the critical path after it
  const int64_t slab_row0 = row_off[kv];
  pdl_wait();
  const int L = len[kv];
  const int per = ((L + kClusterSize - 1) / kClusterSize + kGqTile - 1) / kGqTile * kGqTile;
  const int r_begin = min(L, rank * per), r_end = min(L, r_begin + per);

  __shared__ float cta_o[D];          // this CTA's triple, read by the first CTA of the cluster
  __shared__ float cta_ml[2];
  __shared__ float red[D / 32];
  __shared__ float ring_s[kMaxRecent];

  // self score q . k_new and the new value: only the first CTA needs them; in flight with the stream
  float prod = 0.f, v_self = 0.f;
  if (rank == 0) {
    prod = Elem<T>::load(q + (size_t)slab * D + d) * Elem<T>::load(k_new + (size_t)kv * D + d);
    v_self = Elem<T>::load(v_new + (size_t)kv * D + d);
  }

  if (r_begin < r_end) {              // the same for the whole CTA
    const size_t row0 = (size_t)slab_row0 * kGqRowBytes;
    const GqWarpTriples w = gq_stream_rows<kCmStages>(gq_smem, q + (size_t)slab * D, 1,
                                           reinterpret_cast<const uint8_t *>(k_rows) + row0,
                                           reinterpret_cast<const uint8_t *>(v_rows) + row0, r_begin, r_end, scale_log2);
    float acc, mc, lc;
    gq_combine(w, 0, d, acc, mc, lc);
    cta_o[d] = acc;
    if (d == 0) { cta_ml[0] = mc; cta_ml[1] = lc; }
  } else {
    cta_o[d] = 0.f;
    if (d == 0) { cta_ml[0] = -INFINITY; cta_ml[1] = 0.f; }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) prod += __shfl_xor_sync(0xffffffffu, prod, off);
  if ((d & 31) == 0) red[d >> 5] = prod;
  if (rank == 0) ring_scores<T, D>(rg, kv, q + (size_t)slab * D, scale_log2, ring_s);
  cluster.sync();
  // every CTA of the cluster has read the length and its rows: the new row may go in
  // (never asked for when query heads share a slab: another head's cluster may still be reading its length)
  if (rank == 0) append_new_row<T, D>(ap, kv, L, slab_row0, k_new, v_new);
  if (rank == 0) {
    float s_self = 0.f;
#pragma unroll
    for (int i = 0; i < D / 32; ++i) s_self += red[i];
    s_self *= scale_log2;
    float mr[kClusterSize], lr[kClusterSize], orr[kClusterSize];
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) {
      const float *ml = cluster.map_shared_rank(cta_ml, r);
      mr[r] = ml[0];
      lr[r] = ml[1];
      orr[r] = cluster.map_shared_rank(cta_o, r)[d];
    }
    float mm = s_self;
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) mm = fmaxf(mm, mr[r]);
    for (int r = 0; r < rg.R; ++r) mm = fmaxf(mm, ring_s[r]);
    const float w_self = exp2f(s_self - mm);
    float acc = w_self * v_self;
    float lsum = w_self;
#pragma unroll
    for (int r = 0; r < kClusterSize; ++r) {
      const float w = mr[r] == -INFINITY ? 0.f : exp2f(mr[r] - mm);
      acc = fmaf(w, orr[r], acc);
      lsum = fmaf(w, lr[r], lsum);
    }
    // the evicted tokens of the recent-token window
    for (int r = 0; r < rg.R; ++r) {
      if (ring_s[r] == -INFINITY) continue;
      const float w = exp2f(ring_s[r] - mm);
      acc = fmaf(w, Elem<T>::load(static_cast<const T *>(rg.v) + ((size_t)kv * rg.R + r) * D + d), acc);
      lsum += w;
    }
    Elem<T>::store(out + (size_t)slab * D + d, acc / lsum);
  }
  if (rank == 0 && rg.R > 0 && ap.flag_new != nullptr) {
    // the step carries the append: the new token joins the ring once every thread has read it
    constexpr int kVecs = D * (int)sizeof(T) / 16;
    __syncthreads();
    if (d < kVecs)
      ring_put<kVecs>(rg, kv, d, reinterpret_cast<const uint8_t *>(k_new + (size_t)kv * D),
                      reinterpret_cast<const uint8_t *>(v_new + (size_t)kv * D), ap.flag_new[kv] != 0);
  }
  cluster.sync();
}

static int launch_decode_cluster_mma(int slabs, const void *q, const void *k_new, const void *v_new,
                                     const ag_cache &c, float scale_log2, void *o, const AppendArgs &ap,
                                     const HeadMap &hm, const RecentRing &rg, cudaStream_t st) {
  using T = __nv_bfloat16;
  AG_CUDA_TRY(cudaFuncSetAttribute(decode_cluster_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   gq_smem_bytes(kCmStages)));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kClusterSize, slabs);
  cfg.blockDim = dim3(kGqThreads);
  cfg.dynamicSmemBytes = gq_smem_bytes(kCmStages);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kClusterSize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1] = pdl_attribute();
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_cluster_mma_kernel, static_cast<const T *>(q),
                                 static_cast<const T *>(k_new), static_cast<const T *>(v_new),
                                 static_cast<const T *>(c.k_rows), static_cast<const T *>(c.v_rows),
                                 c.row_off, c.len, scale_log2, static_cast<T *>(o), ap, hm, rg));
  return AG_OK;
}

template <typename T, int D, int kThreads>
static int launch_decode_cluster(int slabs, const void *q, const void *k_new, const void *v_new,
                                 const ag_cache &c, float scale_log2, void *o, const AppendArgs &ap,
                                 const HeadMap &hm, const RecentRing &rg, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kClusterSize, slabs);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kClusterSize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1] = pdl_attribute();
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, decode_cluster_kernel<T, D, kThreads>, static_cast<const T *>(q),
                                 static_cast<const T *>(k_new), static_cast<const T *>(v_new),
                                 static_cast<const T *>(c.k_rows), static_cast<const T *>(c.v_rows),
                                 c.row_off, c.len, scale_log2, static_cast<T *>(o), ap, hm, rg));
  return AG_OK;
}

size_t decode_workspace_bytes(const ag_layer_desc &d) {
  const size_t slabs = (size_t)d.batch * d.heads;
  return align_up(slabs * kMaxSplits * (d.head_dim + 2) * sizeof(float), 256);
}

template <typename T, int D>
static int run_decode(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                      const ag_cache &c, float scale, void *o, void *ws, const AppendArgs &ap, cudaStream_t st) {
  const int slabs = d.batch * d.heads;              // one per (sequence, query head)
  const HeadMap hm{d.heads, kv_heads_of(d)};
  const RecentRing rg = ring_of(d, c);
  const float scale_log2 = scale * 1.4426950408889634f;
  if constexpr (std::is_same_v<T, __nv_bfloat16> && D == kGqD) {
    if (slabs <= kClusterMaxSlabs)
      return launch_decode_cluster_mma(slabs, q, k_new, v_new, c, scale_log2, o, ap, hm, rg, st);
  }
  if (slabs <= kClusterMaxSlabs)
    return launch_decode_cluster<T, D, kClusterThreads>(slabs, q, k_new, v_new, c, scale_log2, o, ap, hm, rg, st);
  int chunk_rows = (c.max_cap + kMaxSplits - 1) / kMaxSplits;
  chunk_rows = (chunk_rows + 127) / 128 * 128;   // whole iterations of the partial kernel (bf16, D = 128)
  const int n_chunks = c.max_cap > 0 ? (c.max_cap + chunk_rows - 1) / chunk_rows : 0;
  float *part_o = static_cast<float *>(ws);
  float *part_ml = part_o + (size_t)slabs * kMaxSplits * D;
  const int group = hm.heads / hm.kv_heads;
  if (n_chunks > 0 && decode_gqa_mma_supported(d)) {
    // grouped-query attention, bf16: the group's heads are the rows of a tensor-core tile
    int rc = launch_decode_partial_gqa_mma(d, q, c, scale_log2, chunk_rows, n_chunks, part_o, part_ml, kMaxSplits, st);
    if (rc) return rc;
  } else if (n_chunks > 0 && (group == 2 || group == 4)) {
    // grouped-query attention: the rows of a key/value slab are read once for its query heads
    dim3 grid(n_chunks, d.batch * hm.kv_heads);
    auto qp = static_cast<const T *>(q);
    auto kr = static_cast<const T *>(c.k_rows), vr = static_cast<const T *>(c.v_rows);
    if (group == 2)
      decode_partial_gqa_kernel<T, D, 2><<<grid, kPartThreads, 0, st>>>(qp, kr, vr, c.row_off, c.len, scale_log2,
                                                                         chunk_rows, part_o, part_ml, hm.kv_heads);
    else
      decode_partial_gqa_kernel<T, D, 4><<<grid, kPartThreads, 0, st>>>(qp, kr, vr, c.row_off, c.len, scale_log2,
                                                                         chunk_rows, part_o, part_ml, hm.kv_heads);
    AG_LAUNCH_CHECK();
  } else if (n_chunks > 0) {
    dim3 grid(n_chunks, slabs);
    decode_partial_kernel<T, D><<<grid, kPartThreads, 0, st>>>(
        static_cast<const T *>(q), static_cast<const T *>(c.k_rows),
        static_cast<const T *>(c.v_rows), c.row_off, c.len, scale_log2, chunk_rows, part_o, part_ml, hm);
    AG_LAUNCH_CHECK();
  }
  decode_combine_kernel<T, D><<<slabs, D, 0, st>>>(
      static_cast<const T *>(q), static_cast<const T *>(k_new), static_cast<const T *>(v_new),
      c.len, scale_log2, chunk_rows, part_o, part_ml, static_cast<T *>(o), c.row_off, ap, hm, rg);
  AG_LAUNCH_CHECK();
  return AG_OK;
}

static int dispatch_decode(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                           const ag_cache &c, float scale, void *o, void *ws, const AppendArgs &ap,
                           cudaStream_t st) {
  if (d.dtype == AG_F32) {
    if (d.head_dim == 64) return run_decode<float, 64>(d, q, k_new, v_new, c, scale, o, ws, ap, st);
    return run_decode<float, 128>(d, q, k_new, v_new, c, scale, o, ws, ap, st);
  }
  if (d.head_dim == 64) return run_decode<__nv_bfloat16, 64>(d, q, k_new, v_new, c, scale, o, ws, ap, st);
  return run_decode<__nv_bfloat16, 128>(d, q, k_new, v_new, c, scale, o, ws, ap, st);
}

int launch_decode(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                  const ag_cache &c, float scale, void *o, void *ws, size_t, cudaStream_t st) {
  return dispatch_decode(d, q, k_new, v_new, c, scale, o, ws, AppendArgs{}, st);
}

// Attention of the step and the conditional append in the same launches.
int launch_decode_step(const ag_layer_desc &d, const void *q, const void *k_new, const void *v_new,
                       const uint8_t *flag_new, const ag_cache &c, float scale, void *o,
                       int32_t *dev_status, void *ws, cudaStream_t st) {
  if (kv_heads_of(d) != d.heads) {
    // query heads share a slab: the append waits for all of them, in a launch of its own
    int rc = dispatch_decode(d, q, k_new, v_new, c, scale, o, ws, AppendArgs{}, st);
    if (rc) return rc;
    return launch_append(d, k_new, v_new, flag_new, c, dev_status, st);
  }
  AppendArgs ap;
  ap.flag_new = flag_new; ap.cap = c.cap; ap.len = c.len;
  ap.k_rows = c.k_rows; ap.v_rows = c.v_rows; ap.dev_status = dev_status;
  return dispatch_decode(d, q, k_new, v_new, c, scale, o, ws, ap, st);
}

// ---------------------------------------------------------------------------
// ag_decode_attn_noalloc: decode attention whose split-K scratch is a fixed
// array inside the library, for callers that cannot obtain device memory.
// ---------------------------------------------------------------------------
constexpr size_t kNoAllocScratchBytes = (size_t)1024 * kMaxSplits * (128 + 2) * sizeof(float);  // 17,039,360

// Lives in the global memory of every GPU that loads the library, until exit.
// Host code may only use this name to look the device address up.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// Device address of g_noalloc_scratch on the CURRENT device, looked up once per device.
static int noalloc_scratch_ptr(void **out) {
  constexpr int kMaxDevices = 64;
  static void *ptrs[kMaxDevices] = {};
  int dev = -1;
  AG_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return AG_ERR_UNSUPPORTED;
  void *p = __atomic_load_n(&ptrs[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    AG_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (!p) return AG_ERR_CUDA;
    __atomic_store_n(&ptrs[dev], p, __ATOMIC_RELEASE);   // same value whichever thread wins
  }
  *out = p;
  return AG_OK;
}

}  // namespace ag

extern "C" int ag_decode_attn_noalloc(const ag_layer_desc *desc, const void *q, const void *k_new,
                                      const void *v_new, const ag_cache *cache, float softmax_scale,
                                      void *o, void *cuda_stream) {
  using namespace ag;
  nvtxRangePushA("ag_decode_attn_noalloc");          // (does nothing unless a profiler is attached)
  struct Pop { ~Pop() { nvtxRangePop(); } } pop_;
  // the same host-side checks as ag_decode_attn, before anything is launched
  int st = check_desc(desc);
  if (st) return st;
  if (!q || !k_new || !v_new || !o) return AG_ERR_INVALID_ARG;
  if (desc->recent_window > 1) return AG_ERR_UNSUPPORTED;     // this entry does not read the ring of recent tokens
  st = check_cache(cache, desc, false);
  if (st) return st;
  if (misaligned16(q) || misaligned16(k_new) || misaligned16(v_new) || misaligned16(o)) return AG_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return AG_ERR_INVALID_ARG;
  // the fixed array bounds the problem size: refuse anything that would not fit
  if (decode_workspace_bytes(*desc) > kNoAllocScratchBytes) return AG_ERR_CAPACITY;
  void *scratch = nullptr;
  st = noalloc_scratch_ptr(&scratch);
  if (st) return st;
  const float scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)desc->head_dim) : softmax_scale;
  // Nothing in the scratch has to start at zero: every partial the merge step
  // reads is written by the chunk pass of this same call.
  return launch_decode(*desc, q, k_new, v_new, *cache, scale, o, scratch, kNoAllocScratchBytes,
                       (cudaStream_t)cuda_stream);
}
