// Per-head stream compaction of K/V by the gate's flags (Sec. 3.3: k_i^(t),
// v_i^(t) are retained iff AG(X)_i^(t) = 1) and the conditional append of the
// decoding stage (Sec. 3.1).
//
//   scan_flags_kernel   one CTA per slab: warp ballot + popc per 32-token
//                       word, shuffle scan across the warps of the CTA,
//                       running carry across 1024-token chunks.
//   gather_rows_kernel  destination-ordered 16-byte-vector row moves: only
//                       retained rows are read, every access is a full row.
#include "ag_common.cuh"

namespace ag {

constexpr int kScanThreads = 1024;

__global__ void __launch_bounds__(kScanThreads)
scan_flags_kernel(const uint8_t *__restrict__ flags, int n, const int32_t *__restrict__ cap,
                  int32_t *__restrict__ len, int32_t *__restrict__ prefix,
                  int32_t *__restrict__ idx, int32_t *__restrict__ dev_status, int check_cap) {
  const int slab = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint8_t *f = flags + (size_t)slab * n;
  int32_t *pre = prefix + (size_t)slab * (n + 1);
  int32_t *ix = idx + (size_t)slab * n;
  __shared__ int warp_excl[32];
  __shared__ int chunk_total;
  int carry = 0;
  for (int base = 0; base < n; base += kScanThreads) {
    const int t = base + threadIdx.x;
    const bool keep = (t < n) && (f[t] != 0);
    const unsigned word = __ballot_sync(0xffffffffu, keep);
    const int in_warp = __popc(word & ((1u << lane) - 1u));
    if (lane == 0) warp_excl[warp] = __popc(word);
    __syncthreads();
    if (warp == 0) {
      const int c = warp_excl[lane];
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += v;
      }
      warp_excl[lane] = inc - c;
      if (lane == 31) chunk_total = inc;
    }
    __syncthreads();
    const int p = carry + warp_excl[warp] + in_warp;
    if (t < n) {
      pre[t] = p;
      if (keep) ix[p] = t;
    }
    carry += chunk_total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    pre[n] = carry;
    if (check_cap && carry > cap[slab]) {
      len[slab] = 0;
      if (dev_status) atomicOr(dev_status, AG_DEV_OVERFLOW);
    } else {
      len[slab] = carry;
    }
  }
}

// One row = D * sizeof(T) bytes = kVecs 16-byte vectors; a group of kVecs
// consecutive lanes moves one row of K and one row of V.
template <int kRowBytes>
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint8_t *__restrict__ K, const uint8_t *__restrict__ V, int n,
                   const int32_t *__restrict__ idx, const int32_t *__restrict__ len,
                   const int64_t *__restrict__ row_off, uint8_t *__restrict__ k_rows,
                   uint8_t *__restrict__ v_rows, int rows_per_cta) {
  constexpr int kVecs = kRowBytes / 16;
  constexpr int kGroups = 256 / kVecs;
  const int slab = blockIdx.y;
  const int L = len[slab];
  const int r0 = blockIdx.x * rows_per_cta;
  if (r0 >= L) return;
  const int r1 = min(L, r0 + rows_per_cta);
  const int g = threadIdx.x / kVecs, v = threadIdx.x % kVecs;
  const int32_t *ix = idx + (size_t)slab * n;
  const uint8_t *Ks = K + (size_t)slab * n * kRowBytes;
  const uint8_t *Vs = V + (size_t)slab * n * kRowBytes;
  const size_t dst0 = (size_t)row_off[slab] * kRowBytes;
  // two rows per group in flight
  for (int r = r0 + g; r < r1; r += 2 * kGroups) {
    const int ra = r, rb = r + kGroups;
    const int ta = ix[ra];
    const bool has_b = rb < r1;
    const int tb = has_b ? ix[rb] : ta;
    uint4 ka = ldg128_stream(Ks + (size_t)ta * kRowBytes + v * 16);
    uint4 va = ldg128_stream(Vs + (size_t)ta * kRowBytes + v * 16);
    uint4 kb = ldg128_stream(Ks + (size_t)tb * kRowBytes + v * 16);
    uint4 vb = ldg128_stream(Vs + (size_t)tb * kRowBytes + v * 16);
    *reinterpret_cast<uint4 *>(k_rows + dst0 + (size_t)ra * kRowBytes + v * 16) = ka;
    *reinterpret_cast<uint4 *>(v_rows + dst0 + (size_t)ra * kRowBytes + v * 16) = va;
    if (has_b) {
      *reinterpret_cast<uint4 *>(k_rows + dst0 + (size_t)rb * kRowBytes + v * 16) = kb;
      *reinterpret_cast<uint4 *>(v_rows + dst0 + (size_t)rb * kRowBytes + v * 16) = vb;
    }
  }
}

template <int kRowBytes>
__global__ void __launch_bounds__(256)
append_rows_kernel(const uint8_t *__restrict__ k_new, const uint8_t *__restrict__ v_new,
                   const uint8_t *__restrict__ flag_new, int n_slabs,
                   const int64_t *__restrict__ row_off, const int32_t *__restrict__ cap,
                   int32_t *__restrict__ len, uint8_t *__restrict__ k_rows,
                   uint8_t *__restrict__ v_rows, int32_t *__restrict__ dev_status) {
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
}

static int row_bytes(const ag_layer_desc &d) {
  return d.head_dim * (d.dtype == AG_F32 ? 4 : 2);
}

size_t compact_workspace_bytes(const ag_layer_desc &d) {
  // room for idx when the caller does not want it back
  return align_up((size_t)d.batch * d.heads * d.seq * sizeof(int32_t), 256);
}

int launch_compact(const ag_layer_desc &d, const void *K, const void *V, const uint8_t *flags,
                   const ag_cache &c, int32_t *prefix, int32_t *idx, int32_t *dev_status,
                   void *ws, cudaStream_t st) {
  const int slabs = d.batch * d.heads;
  int32_t *ix = idx ? idx : static_cast<int32_t *>(ws);
  scan_flags_kernel<<<slabs, kScanThreads, 0, st>>>(flags, d.seq, c.cap, c.len, prefix, ix,
                                                    dev_status, K != nullptr);
  AG_LAUNCH_CHECK();
  if (!K) return AG_OK;
  const int rb = row_bytes(d);
  const int rows_per_cta = 128;
  dim3 grid((d.seq + rows_per_cta - 1) / rows_per_cta, slabs);
  auto Kb = static_cast<const uint8_t *>(K);
  auto Vb = static_cast<const uint8_t *>(V);
  auto kr = static_cast<uint8_t *>(c.k_rows);
  auto vr = static_cast<uint8_t *>(c.v_rows);
  switch (rb) {
    case 128:
      gather_rows_kernel<128><<<grid, 256, 0, st>>>(Kb, Vb, d.seq, ix, c.len, c.row_off, kr, vr, rows_per_cta);
      break;
    case 256:
      gather_rows_kernel<256><<<grid, 256, 0, st>>>(Kb, Vb, d.seq, ix, c.len, c.row_off, kr, vr, rows_per_cta);
      break;
    case 512:
      gather_rows_kernel<512><<<grid, 256, 0, st>>>(Kb, Vb, d.seq, ix, c.len, c.row_off, kr, vr, rows_per_cta);
      break;
    default:
      return AG_ERR_UNSUPPORTED;
  }
  AG_LAUNCH_CHECK();
  return AG_OK;
}

int launch_append(const ag_layer_desc &d, const void *k_new, const void *v_new,
                  const uint8_t *flag_new, const ag_cache &c, int32_t *dev_status,
                  cudaStream_t st) {
  const int slabs = d.batch * d.heads;
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
  switch (rb) {
    case 128:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<128>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status));
      break;
    case 256:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<256>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status));
      break;
    case 512:
      AG_CUDA_TRY(cudaLaunchKernelEx(&cfg, append_rows_kernel<512>, kn, vn, flag_new, slabs, c.row_off, c.cap, c.len, kr, vr, dev_status));
      break;
    default:
      return AG_ERR_UNSUPPORTED;
  }
  AG_LAUNCH_CHECK();
  return AG_OK;
}

}  // namespace ag
