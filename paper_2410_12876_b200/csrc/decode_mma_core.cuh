// Core of decode attention on warp-level MMAs: rows [r_begin, r_end) of one key/value slab against
// the G <= 16 query vectors that read it (G query heads of a group, or one head), streamed through
// shared memory.  Used by the chunk pass of grouped-query decode and by the cluster form of decode.
//
// The G queries are the rows of a 16-row MMA operand (the other rows are zero): m16n8k16 bf16 MMAs,
// the shape that fits an M of 1..16 (a tcgen05 tile needs M >= 64); the contraction is bound by
// memory, and what the tensor cores buy is fewer instructions per row, not FLOP/s.  Rows go global ->
// shared by 16-byte cp.async in tiles of 64 rows (K and V; the next tile is in flight while one is
// worked on); each of the four warps owns 16 rows of every tile and keeps its own running softmax;
// the warps' (m, l, o) triples end in shared memory and gq_combine() merges them.
#pragma once
#include "ag_common.cuh"
#include "mma_sync.cuh"

namespace ag {

constexpr int kGqD = 128;                 // head_dim (bf16)
constexpr int kGqWarps = 4, kGqThreads = kGqWarps * 32;
constexpr int kGqTile = kGqWarps * 16;    // rows per tile: 16 per warp
constexpr int kGqRowBytes = kGqD * 2;
constexpr int kGqTileBytes = kGqTile * kGqRowBytes;           // 16 KB
// dynamic shared memory of a kernel that streams with a ring of `stages` (K tile, V tile) pairs
constexpr int gq_smem_bytes(int stages) { return stages * 2 * kGqTileBytes; }
constexpr int kGqMaxGroup = 16;

// Per-warp triples in shared memory, laid over the tile ring once the rows have been consumed.
struct GqWarpTriples {
  float *o, *m, *l;     // [warps][16][D], [warps][16], [warps][16]
};

// Every thread of the CTA (kGqThreads of them) calls this with the same arguments; r_begin < r_end.
// q: G consecutive query vectors [G][D]; Kg, Vg: first row of the slab.  Returns after a CTA barrier
// with the warps' triples in shared memory (gq_smem: gq_smem_bytes(kGqStages) of dynamic shared memory;
// kGqStages - 1 tiles are in flight while one is worked on).
template <int kGqStages>
__device__ __forceinline__ GqWarpTriples gq_stream_rows(uint8_t *gq_smem, const __nv_bfloat16 *__restrict__ q, int G,
                                                        const uint8_t *__restrict__ Kg, const uint8_t *__restrict__ Vg,
                                                        int r_begin, int r_end, float scale_log2) {
  const int n_tiles = (r_end - r_begin + kGqTile - 1) / kGqTile;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;                                       // fragment row, column pair
  const uint32_t smem0 = (uint32_t)__cvta_generic_to_shared(gq_smem);

  // tile i -> stage i % kGqStages; rows past r_end are clamped to the last valid row (weight 0 below)
  auto load_tile = [&](int i) {
    const uint32_t sk = smem0 + (i % kGqStages) * 2 * kGqTileBytes, sv = sk + kGqTileBytes;
    const int r0 = r_begin + i * kGqTile;
#pragma unroll
    for (int x = 0; x < kGqTile * 16 / kGqThreads; ++x) {
      const int idx = threadIdx.x + x * kGqThreads, r = idx >> 4, c = idx & 15;
      const size_t src = (size_t)min(r0 + r, r_end - 1) * kGqRowBytes + c * 16;
      cp_async16(sk + tile256_off(r, c), Kg + src);
      cp_async16(sv + tile256_off(r, c), Vg + src);
    }
  };
#pragma unroll
  for (int i = 0; i < kGqStages - 1; ++i) {
    if (i < n_tiles) load_tile(i);
    cp_async_commit();
  }

  // A fragments of Q: row g = query head g of the group (rows >= G are zero), 8 steps of 16 dims
  uint32_t qa[kGqD / 16][4];
#pragma unroll
  for (int ks = 0; ks < kGqD / 16; ++ks) {
    const uint32_t *qrow = reinterpret_cast<const uint32_t *>(q + (size_t)min(g, G - 1) * kGqD);
    const uint32_t lo = qrow[ks * 8 + t], hi = qrow[ks * 8 + 4 + t];
    qa[ks][0] = g < G ? lo : 0u;
    qa[ks][1] = 0u;                                     // rows 8..15: G <= 8 is all this kernel is asked for
    qa[ks][2] = g < G ? hi : 0u;
    qa[ks][3] = 0u;
  }
  const bool two_halves = G > 8;
  if (two_halves) {
#pragma unroll
    for (int ks = 0; ks < kGqD / 16; ++ks) {
      const uint32_t *qrow = reinterpret_cast<const uint32_t *>(q + (size_t)min(g + 8, G - 1) * kGqD);
      qa[ks][1] = g + 8 < G ? qrow[ks * 8 + t] : 0u;
      qa[ks][3] = g + 8 < G ? qrow[ks * 8 + 4 + t] : 0u;
    }
  }

  float o[kGqD / 8][4];
#pragma unroll
  for (int nt = 0; nt < kGqD / 8; ++nt)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[nt][e] = 0.f;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};       // rows g and g + 8

  for (int i = 0; i < n_tiles; ++i) {
    if (i + kGqStages - 1 < n_tiles) load_tile(i + kGqStages - 1);
    cp_async_commit();
    cp_async_wait<kGqStages - 1>();                             // tile i has landed (this thread's pieces)
    __syncthreads();                                            // ... and everybody's
    const uint32_t sk = smem0 + (i % kGqStages) * 2 * kGqTileBytes, sv = sk + kGqTileBytes;
    const int key0 = r_begin + i * kGqTile + warp * 16;         // this warp's 16 rows of the tile

    if (key0 < r_end) {
      // S = Q K^T for 16 keys: two 8-key column tiles
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < kGqD / 16; ++ks) {
        uint32_t b[4];
        // matrices: (keys 0-7, dims lo), (keys 0-7, dims hi), (keys 8-15, dims lo), (keys 8-15, dims hi)
        const int mi = lane >> 3, row = warp * 16 + (mi >> 1) * 8 + (lane & 7);
        ldmatrix_x4(b, sk + tile256_off(row, ks * 2 + (mi & 1)));
        mma_16816(s0, qa[ks], b[0], b[1]);
        mma_16816(s1, qa[ks], b[2], b[3]);
      }
      // online softmax of rows g (and g + 8): this thread holds keys 2t, 2t+1 of each column tile
      uint32_t pa[4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float sv4[4] = {s0[2 * h], s0[2 * h + 1], s1[2 * h], s1[2 * h + 1]};
        const int kcol[4] = {2 * t, 2 * t + 1, 8 + 2 * t, 9 + 2 * t};
        float tmax = -INFINITY;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          sv4[e] = (key0 + kcol[e] < r_end) ? sv4[e] * scale_log2 : -INFINITY;
          tmax = fmaxf(tmax, sv4[e]);
        }
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        const float m_new = fmaxf(m[h], tmax);                  // finite: key0 < r_end, so column 0 is valid
        const float alpha = exp2f(m[h] - m_new);                // m = -inf at first: 0
        float p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) p[e] = exp2f(sv4[e] - m_new);
        const bool row_used = h == 0 ? g < G : g + 8 < G;       // unused rows: zero weights, not 2^(0 - m)
        l[h] = l[h] * alpha + (row_used ? (p[0] + p[1]) + (p[2] + p[3]) : 0.f);
        m[h] = m_new;
        pa[h] = row_used ? pack2_bf16(p[0], p[1]) : 0u;
        pa[2 + h] = row_used ? pack2_bf16(p[2], p[3]) : 0u;
#pragma unroll
        for (int nt = 0; nt < kGqD / 8; ++nt) {
          o[nt][2 * h] *= alpha;
          o[nt][2 * h + 1] *= alpha;
        }
      }
      // O += P V: 16 keys x 128 dims, two 8-dim column tiles per ldmatrix
#pragma unroll
      for (int nt2 = 0; nt2 < kGqD / 16; ++nt2) {
        uint32_t b[4];
        // matrices: (keys 0-7, dims lo), (keys 8-15, dims lo), (keys 0-7, dims hi), (keys 8-15, dims hi)
        const int mi = lane >> 3, row = warp * 16 + (mi & 1) * 8 + (lane & 7);
        ldmatrix_x4_trans(b, sv + tile256_off(row, nt2 * 2 + (mi >> 1)));
        mma_16816(o[2 * nt2], pa, b[0], b[1]);
        mma_16816(o[2 * nt2 + 1], pa, b[2], b[3]);
      }
    }
    __syncthreads();                                            // the stage may be refilled
  }
  cp_async_wait<0>();

  // merge the four warps' triples through shared memory (the tiles are no longer needed)
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l[h] += __shfl_xor_sync(0xffffffffu, l[h], 1);
    l[h] += __shfl_xor_sync(0xffffffffu, l[h], 2);
  }
  float *sm_o = reinterpret_cast<float *>(gq_smem);             // [warps][16][D]
  float *sm_m = sm_o + kGqWarps * kGqMaxGroup * kGqD;           // [warps][16]
  float *sm_l = sm_m + kGqWarps * kGqMaxGroup;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int row = g + 8 * h;
    if (row < G) {
#pragma unroll
      for (int nt = 0; nt < kGqD / 8; ++nt) {
        float *dst = sm_o + ((size_t)(warp * kGqMaxGroup + row)) * kGqD + nt * 8 + 2 * t;
        dst[0] = o[nt][2 * h];
        dst[1] = o[nt][2 * h + 1];
      }
      if (t == 0) {
        sm_m[warp * kGqMaxGroup + row] = m[h];
        sm_l[warp * kGqMaxGroup + row] = l[h];
      }
    }
  }
  __syncthreads();
  return GqWarpTriples{sm_o, sm_m, sm_l};
}

// The CTA's triple for query h, output dimension d, from the warps' triples.
__device__ __forceinline__ void gq_combine(const GqWarpTriples &w, int h, int d, float &acc, float &mc, float &lc) {
  mc = -INFINITY;
#pragma unroll
  for (int i = 0; i < kGqWarps; ++i) mc = fmaxf(mc, w.m[i * kGqMaxGroup + h]);
  acc = 0.f;
  lc = 0.f;
#pragma unroll
  for (int i = 0; i < kGqWarps; ++i) {
    const float mw = w.m[i * kGqMaxGroup + h];
    const float wgt = mw == -INFINITY ? 0.f : exp2f(mw - mc);
    acc = fmaf(wgt, w.o[((size_t)(i * kGqMaxGroup + h)) * kGqD + d], acc);
    lc = fmaf(wgt, w.l[i * kGqMaxGroup + h], lc);
  }
}

}  // namespace ag
