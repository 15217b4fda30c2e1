// Per-head stream compaction of K/V by the gate's flags (Sec. 3.3: k_i^(t),
// v_i^(t) are retained iff AG(X)_i^(t) = 1) and the conditional append of the
// decoding stage (Sec. 3.1).
//
//   compact_kernel   one CTA per 256 tokens of a slab.  It counts the flags of the whole slab row
//                    (a few KB, read as 16-byte vectors) to get the number of retained tokens
//                    before its chunk and in the slab, ranks its own tokens by warp ballot +
//                    popc, writes prefix and idx for them, and moves the retained rows of its
//                    chunk: 16-byte-vector row moves, only retained rows are read, every access
//                    is a full row.  One launch; no pass over the flags on its own.
#include "ag_common.cuh"

namespace ag {

constexpr int kCompactThreads = 256;   // = tokens per CTA

// Bytes of a 32-bit word that are not zero.
__device__ __forceinline__ int nonzero_bytes(uint32_t w) { return __popc(__vcmpne4(w, 0u) & 0x01010101u); }

// One row = D * sizeof(T) bytes = kVecs 16-byte vectors; a group of kVecs consecutive lanes moves
// one row of K and one row of V.  kRowBytes = 0: count pass, no rows move.
template <int kRowBytes>
__global__ void __launch_bounds__(kCompactThreads)
compact_kernel(const uint8_t *__restrict__ flags, int n, const int32_t *__restrict__ cap,
               int32_t *__restrict__ len, int32_t *__restrict__ prefix, int32_t *__restrict__ idx,
               int32_t *__restrict__ dev_status, const uint8_t *__restrict__ K,
               const uint8_t *__restrict__ V, const int64_t *__restrict__ row_off,
               uint8_t *__restrict__ k_rows, uint8_t *__restrict__ v_rows) {
  const int slab = blockIdx.y, t0 = blockIdx.x * kCompactThreads;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint8_t *f = flags + (size_t)slab * n;
  __shared__ int red_before[kCompactThreads / 32], red_total[kCompactThreads / 32];
  __shared__ int warp_excl[kCompactThreads / 32];
  __shared__ int tok_list[kCompactThreads];

  // retained tokens before this chunk, and in the slab
  int before = 0, total = 0;
  if ((n & 15) == 0) {                       // rows of the flag array start on 16-byte boundaries
    const uint4 *fv = reinterpret_cast<const uint4 *>(f);
    for (int x = threadIdx.x; x < n / 16; x += kCompactThreads) {
      const uint4 w = ldg128(fv + x);
      const int c = nonzero_bytes(w.x) + nonzero_bytes(w.y) + nonzero_bytes(w.z) + nonzero_bytes(w.w);
      total += c;
      if (x * 16 < t0) before += c;          // t0 is a multiple of 16: a vector lies on one side
    }
  } else {
    for (int x = threadIdx.x; x < n; x += kCompactThreads) {
      const int c = f[x] != 0;
      total += c;
      if (x < t0) before += c;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    before += __shfl_xor_sync(0xffffffffu, before, o);
    total += __shfl_xor_sync(0xffffffffu, total, o);
  }
  // this chunk's tokens
  const int t = t0 + threadIdx.x;
  const bool keep = (t < n) && (f[t] != 0);
  const unsigned word = __ballot_sync(0xffffffffu, keep);
  const int in_warp = __popc(word & ((1u << lane) - 1u));
  if (lane == 0) { red_before[warp] = before; red_total[warp] = total; warp_excl[warp] = __popc(word); }
  __syncthreads();
  before = 0; total = 0;
  int excl = 0, count = 0;
#pragma unroll
  for (int w = 0; w < kCompactThreads / 32; ++w) {
    before += red_before[w];
    total += red_total[w];
    if (w < warp) excl += warp_excl[w];
    count += warp_excl[w];
  }
  const int local = excl + in_warp;          // rank within the chunk
  const int p = before + local;              // rank within the slab
  int32_t *pre = prefix + (size_t)slab * (n + 1);
  if (t < n) {
    pre[t] = p;
    if (keep) {
      idx[(size_t)slab * n + p] = t;
      tok_list[local] = t;
    }
  }
  const bool overflow = kRowBytes != 0 && total > cap[slab];
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    pre[n] = total;
    len[slab] = overflow ? 0 : total;
    if (overflow && dev_status) atomicOr(dev_status, AG_DEV_OVERFLOW);
  }
  if (kRowBytes == 0 || overflow) return;    // count pass, or a slab that does not fit: nothing moves
  __syncthreads();

  constexpr int kVecs = kRowBytes > 0 ? kRowBytes / 16 : 1;
  constexpr int kGroups = kCompactThreads / kVecs;
  const int g = threadIdx.x / kVecs, v = threadIdx.x % kVecs;
  const uint8_t *Ks = K + (size_t)slab * n * kRowBytes;
  const uint8_t *Vs = V + (size_t)slab * n * kRowBytes;
  const size_t dst0 = ((size_t)row_off[slab] + before) * kRowBytes;
  // kFlight rows of K and of V per group in flight
  constexpr int kFlight = 4;
  for (int j = g; j < count; j += kFlight * kGroups) {
    uint4 kv[kFlight], vv[kFlight];
#pragma unroll
    for (int u = 0; u < kFlight; ++u) {
      const int tu = tok_list[min(j + u * kGroups, count - 1)];
      kv[u] = ldg128_stream(Ks + (size_t)tu * kRowBytes + v * 16);
      vv[u] = ldg128_stream(Vs + (size_t)tu * kRowBytes + v * 16);
    }
#pragma unroll
    for (int u = 0; u < kFlight; ++u) {
      const int ju = j + u * kGroups;
      if (ju < count) {
        *reinterpret_cast<uint4 *>(k_rows + dst0 + (size_t)ju * kRowBytes + v * 16) = kv[u];
        *reinterpret_cast<uint4 *>(v_rows + dst0 + (size_t)ju * kRowBytes + v * 16) = vv[u];
      }
    }
  }
}

template <int kRowBytes>
__global__ void __launch_bounds__(256)
append_rows_kernel(const uint8_t *__restrict__ k_new, const uint8_t *__restrict__ v_new,
                   const uint8_t *__restrict__ flag_new, int n_slabs,
                   const int64_t *__restrict__ row_off, const int32_t *__restrict__ cap,
                   int32_t *__restrict__ len, uint8_t *__restrict__ k_rows,
                   uint8_t *__restrict__ v_rows, int32_t *__restrict__ dev_status, const RecentRing ring) {
  constexpr int kVecs = kRowBytes / 16;
  constexpr int kGroups = 256 / kVecs;
  const int slab = blockIdx.x * kGroups + threadIdx.x / kVecs;
  const int v = threadIdx.x % kVecs;
  pdl_launch_dependents();
  pdl_wait();
  const bool want = slab < n_slabs && flag_new[slab] != 0;
  // every lane of a group reads the length before lane 0 of the group bumps it
  const int L = want ? len[slab] : 0;
  const bool full = want && L >= cap[slab];
  __syncwarp();
  if (want && !full) {
    const size_t dst = ((size_t)row_off[slab] + L) * kRowBytes + v * 16;
    const size_t src = (size_t)slab * kRowBytes + v * 16;
    *reinterpret_cast<uint4 *>(k_rows + dst) = *reinterpret_cast<const uint4 *>(k_new + src);
    *reinterpret_cast<uint4 *>(v_rows + dst) = *reinterpret_cast<const uint4 *>(v_new + src);
    if (v == 0) len[slab] = L + 1;
  }
  if (full && v == 0 && dev_status) atomicOr(dev_status, AG_DEV_OVERFLOW);
  // recent-token window: kept or not, the token is one of the slab's recent tokens from now on
  if (ring.R > 0 && slab < n_slabs)
    ring_put<kVecs>(ring, slab, v, k_new + (size_t)slab * kRowBytes, v_new + (size_t)slab * kRowBytes, want);
}

// Recent-token window: after the prompt, the ring of a slab holds its last R tokens (token t in
// slot t % R), the evicted ones marked live; a prompt shorter than R leaves the other slots dead.
// With per-sequence lengths the prompt of a slab is the first seq_lens[b] of its n positions.
// One CTA per slab, thread (slot, 16-byte piece).
template <int kRowBytes>
__global__ void recent_fill_kernel(const uint8_t *__restrict__ K, const uint8_t *__restrict__ V,
                                   const uint8_t *__restrict__ flags, int n, const int32_t *__restrict__ seq_lens,
                                   int kv_heads, const RecentRing ring) {
  constexpr int kVecs = kRowBytes / 16;
  const int slab = blockIdx.x, slot = threadIdx.x / kVecs, v = threadIdx.x % kVecs;
  if (slot >= ring.R) return;
  const int len = seq_lens ? min(max(seq_lens[slab / kv_heads], 0), n) : n;   // tokens of this slab's prompt
  // the last token whose number is slot modulo R, if the prompt has one
  const bool have = slot <= len - 1;
  const int t = have ? slot + (len - 1 - slot) / ring.R * ring.R : 0;
  if (have) {
    const size_t src = ((size_t)slab * n + t) * kRowBytes + v * 16;
    const size_t dst = ((size_t)slab * ring.R + slot) * kRowBytes + v * 16;
    *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(ring.k) + dst) = *reinterpret_cast<const uint4 *>(K + src);
    *reinterpret_cast<uint4 *>(static_cast<uint8_t *>(ring.v) + dst) = *reinterpret_cast<const uint4 *>(V + src);
  }
  if (v == 0) ring.live[(size_t)slab * ring.R + slot] = (have && flags[(size_t)slab * n + t] == 0) ? 1 : 0;
  if (threadIdx.x == 0) ring.pos[slab] = len;
}

static int row_bytes(const ag_layer_desc &d) {
  return d.head_dim * (d.dtype == AG_F32 ? 4 : 2);
}

size_t compact_workspace_bytes(const ag_layer_desc &d) {
  // room for idx when the caller does not want it back
  return align_up((size_t)d.batch * kv_heads_of(d) * d.seq * sizeof(int32_t), 256);
}

int launch_compact(const ag_layer_desc &d, const void *K, const void *V, const uint8_t *flags,
                   const ag_cache &c, int32_t *prefix, int32_t *idx, int32_t *dev_status,
                   void *ws, cudaStream_t st) {
  const int slabs = d.batch * kv_heads_of(d);
  int32_t *ix = idx ? idx : static_cast<int32_t *>(ws);
  dim3 grid((d.seq + kCompactThreads - 1) / kCompactThreads, slabs);
  auto Kb = static_cast<const uint8_t *>(K);
  auto Vb = static_cast<const uint8_t *>(V);
  auto kr = static_cast<uint8_t *>(c.k_rows);
  auto vr = static_cast<uint8_t *>(c.v_rows);
  switch (K ? row_bytes(d) : 0) {
    case 0:
      compact_kernel<0><<<grid, kCompactThreads, 0, st>>>(flags, d.seq, c.cap, c.len, prefix, ix, dev_status, Kb, Vb, c.row_off, kr, vr);
      break;
    case 128:
      compact_kernel<128><<<grid, kCompactThreads, 0, st>>>(flags, d.seq, c.cap, c.len, prefix, ix, dev_status, Kb, Vb, c.row_off, kr, vr);
      break;
    case 256:
      compact_kernel<256><<<grid, kCompactThreads, 0, st>>>(flags, d.seq, c.cap, c.len, prefix, ix, dev_status, Kb, Vb, c.row_off, kr, vr);
      break;
    case 512:
      compact_kernel<512><<<grid, kCompactThreads, 0, st>>>(flags, d.seq, c.cap, c.len, prefix, ix, dev_status, Kb, Vb, c.row_off, kr, vr);
      break;
    default:
      return AG_ERR_UNSUPPORTED;
  }
  AG_LAUNCH_CHECK();
  const RecentRing ring = ring_of(d, c);
  if (K && ring.R > 0) return launch_recent_fill(d, K, V, flags, c, st);
  return AG_OK;
}

// Ring of a recent-token window from the dense K, V of the prompt (one more small launch).
int launch_recent_fill(const ag_layer_desc &d, const void *K, const void *V, const uint8_t *flags, const ag_cache &c,
                       cudaStream_t st) {
  const RecentRing ring = ring_of(d, c);
  if (ring.R == 0) return AG_OK;
  const int slabs = d.batch * kv_heads_of(d);
  auto Kb = static_cast<const uint8_t *>(K);
  auto Vb = static_cast<const uint8_t *>(V);
  const int threads = ring.R * (row_bytes(d) / 16);
  switch (row_bytes(d)) {
    case 128: recent_fill_kernel<128><<<slabs, threads, 0, st>>>(Kb, Vb, flags, d.seq, d.seq_lens, kv_heads_of(d), ring); break;
    case 256: recent_fill_kernel<256><<<slabs, threads, 0, st>>>(Kb, Vb, flags, d.seq, d.seq_lens, kv_heads_of(d), ring); break;
    default: recent_fill_kernel<512><<<slabs, threads, 0, st>>>(Kb, Vb, flags, d.seq, d.seq_lens, kv_heads_of(d), ring); break;
  }
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int launch_append(const ag_layer_desc &d, const void *k_new, const void *v_new,
                  const uint8_t *flag_new, const ag_cache &c, int32_t *dev_status,
                  cudaStream_t st) {
  const int slabs = d.batch * kv_heads_of(d);
  const int rb = row_bytes(d);
  auto kn = static_cast<const uint8_t *>(k_new);
  auto vn = static_cast<const uint8_t *>(v_new);
  auto kr = static_cast<uint8_t *>(c.k_rows);
  auto vr = static_cast<uint8_t *>(c.v_rows);
  const int groups = 256 / (rb / 16);
  const int grid = (slabs + groups - 1) / groups;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(256);
  cfg.stream = st;
  cudaLaunchAttribute attr = pdl_attribute();
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  const RecentRing ring = ring_of(d, c);
  switch (rb) {
    case 128:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<128>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status, ring));
      break;
    case 256:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<256>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status, ring));
      break;
    case 512:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<512>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status, ring));
      break;
    default:
      return AG_ERR_UNSUPPORTED;
  }
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace ag
