// C boundary of the AG-gated attention layer: argument checks and dispatch.
// Every check that can be made on the host is made here, before any launch.
#include <math.h>
#include <nvtx3/nvToolsExt.h>

#include "ag_common.cuh"

namespace ag {
static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

static bool dim_ok(int d) { return d == 64 || d == 128; }

// Checks of the fields every call uses.
int check_desc(const ag_layer_desc *d) {
  if (!d) return AG_ERR_INVALID_ARG;
  if (d->batch <= 0 || d->seq <= 0 || d->heads <= 0) return AG_ERR_INVALID_ARG;
  if (d->dtype != AG_F32 && d->dtype != AG_BF16) return AG_ERR_INVALID_ARG;
  if (!dim_ok(d->head_dim)) return AG_ERR_UNSUPPORTED;
  if ((int64_t)d->batch * d->heads > (int64_t)1 << 24) return AG_ERR_UNSUPPORTED;
  if (d->kv_heads < 0 || (d->kv_heads > 0 && d->heads % d->kv_heads != 0)) return AG_ERR_INVALID_ARG;
  if (d->recent_window < 0) return AG_ERR_INVALID_ARG;
  if (d->recent_window > kMaxRecent + 1) return AG_ERR_UNSUPPORTED;
  return AG_OK;
}

// Checks of the gate fields (Sec. 3.3 requires h' < h).
static int check_gate_desc(const ag_layer_desc *d) {
  int st = check_desc(d);
  if (st) return st;
  if (d->hidden <= 0 || d->gate_heads <= 0) return AG_ERR_INVALID_ARG;
  if (d->gate_heads >= d->heads) return AG_ERR_INVALID_ARG;
  if (!(d->tau > 0.f && d->tau < 1.f)) return AG_ERR_INVALID_ARG;
  if (d->gate_causal != 0 && d->gate_causal != 1) return AG_ERR_INVALID_ARG;
  if (!dim_ok(d->gate_head_dim)) return AG_ERR_UNSUPPORTED;
  if (d->hidden % 8 != 0) return AG_ERR_UNSUPPORTED;
  return AG_OK;
}

// need_recent: the call reads or writes the ring of recent tokens (compaction, decode, append).
int check_cache(const ag_cache *c, const ag_layer_desc *d, bool need_recent) {
  if (!c) return AG_ERR_INVALID_ARG;
  if (need_recent && d && recent_rows(*d) > 0) {
    if (!c->recent_k || !c->recent_v || !c->recent_live || !c->pos) return AG_ERR_INVALID_ARG;
    if (misaligned16(c->recent_k) || misaligned16(c->recent_v)) return AG_ERR_INVALID_ARG;
  }
  if (!c->row_off || !c->cap || !c->len) return AG_ERR_INVALID_ARG;
  if (c->pool_rows < 0 || c->max_cap < 0) return AG_ERR_INVALID_ARG;
  if (c->pool_rows > 0 && (!c->k_rows || !c->v_rows)) return AG_ERR_INVALID_ARG;
  if (misaligned16(c->k_rows) || misaligned16(c->v_rows)) return AG_ERR_INVALID_ARG;
  if (c->max_cap > c->pool_rows) return AG_ERR_CAPACITY;
  return AG_OK;
}

static int check_ws(size_t need, void *ws, size_t ws_bytes) {
  if (need == 0) return AG_OK;
  if (!ws || ws_bytes < need) return AG_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(ws) & 255u) return AG_ERR_WORKSPACE;
  return AG_OK;
}
}  // namespace ag

using namespace ag;

namespace {
// A named range around every call of the boundary, for timelines: the header-only NVTX layer does
// nothing (one predictable branch) unless a profiler has attached itself to the process.
struct CallRange {
  explicit CallRange(const char *name) { nvtxRangePushA(name); }
  ~CallRange() { nvtxRangePop(); }
};
}  // namespace

extern "C" {

size_t ag_workspace_bytes(const ag_layer_desc *desc, int which) {
  switch (which) {
    case AG_CALL_GATE:
      return check_gate_desc(desc) ? 0 : gate_workspace_bytes(*desc);
    case AG_CALL_COMPACT:
      return check_desc(desc) ? 0 : compact_workspace_bytes(*desc);
    case AG_CALL_PREFILL:
      return check_desc(desc) ? 0 : prefill_workspace_bytes(*desc);
    case AG_CALL_DECODE:
      return check_desc(desc) ? 0 : decode_workspace_bytes(*desc);
    default:
      return 0;
  }
}

int ag_gate_forward(const ag_layer_desc *desc, const void *X, const void *Wq_g,
                    const void *Wk_g, const void *Wv_g, const void *Wo_g,
                    const float *gamma, float *scores, uint8_t *flags, void *ws,
                    size_t ws_bytes, void *cuda_stream) {
  CallRange range_("ag_gate_forward");
  int st = check_gate_desc(desc);
  if (st) return st;
  if (!X || !Wq_g || !Wk_g || !Wv_g || !Wo_g || !flags) return AG_ERR_INVALID_ARG;
  if (misaligned16(X) || misaligned16(Wq_g) || misaligned16(Wk_g) || misaligned16(Wv_g) ||
      misaligned16(Wo_g) || misaligned16(flags) || misaligned16(scores) || misaligned16(gamma))
    return AG_ERR_INVALID_ARG;
  st = check_ws(gate_workspace_bytes(*desc), ws, ws_bytes);
  if (st) return st;
  return launch_gate(*desc, X, Wq_g, Wk_g, Wv_g, Wo_g, gamma, scores, flags, ws,
                     (cudaStream_t)cuda_stream);
}

int ag_gate_linear_forward(const ag_layer_desc *desc, const void *X, const void *W_lin,
                           const float *gamma, float *scores, uint8_t *flags, void *cuda_stream) {
  CallRange range_("ag_gate_linear_forward");
  int st = check_desc(desc);
  if (st) return st;
  if (desc->hidden <= 0 || !(desc->tau > 0.f && desc->tau < 1.f)) return AG_ERR_INVALID_ARG;
  if (!X || !W_lin || !flags) return AG_ERR_INVALID_ARG;
  if (misaligned16(X) || misaligned16(W_lin) || misaligned16(flags) || misaligned16(scores) || misaligned16(gamma))
    return AG_ERR_INVALID_ARG;
  return launch_gate_linear(*desc, X, W_lin, gamma, scores, flags, (cudaStream_t)cuda_stream);
}

int ag_compact_kv(const ag_layer_desc *desc, const void *K, const void *V,
                  const uint8_t *flags, ag_cache *cache, int32_t *prefix,
                  int32_t *idx, int32_t *dev_status, void *ws, size_t ws_bytes,
                  void *cuda_stream) {
  CallRange range_("ag_compact_kv");
  int st = check_desc(desc);
  if (st) return st;
  if (!flags || !prefix) return AG_ERR_INVALID_ARG;
  if ((K == nullptr) != (V == nullptr)) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, K != nullptr);
  if (st) return st;
  if (misaligned16(K) || misaligned16(V) || misaligned16(flags) || misaligned16(prefix) ||
      misaligned16(idx))
    return AG_ERR_INVALID_ARG;
  if (!idx) {
    st = check_ws(compact_workspace_bytes(*desc), ws, ws_bytes);
    if (st) return st;
  }
  return launch_compact(*desc, K, V, flags, *cache, prefix, idx, dev_status, ws,
                        (cudaStream_t)cuda_stream);
}

int ag_kv_project_cache(const ag_layer_desc *desc, const void *X, const void *Wk, const void *Wv,
                        const uint8_t *flags, ag_cache *cache, int32_t *prefix, int32_t *idx, void *K, void *V,
                        int32_t *dev_status, void *cuda_stream) {
  CallRange range_("ag_kv_project_cache");
  int st = check_desc(desc);
  if (st) return st;
  if (desc->hidden <= 0) return AG_ERR_INVALID_ARG;
  if (!X || !Wk || !Wv || !flags || !prefix || !K || !V) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, true);
  if (st) return st;
  if (misaligned16(X) || misaligned16(Wk) || misaligned16(Wv) || misaligned16(K) || misaligned16(V) ||
      misaligned16(flags) || misaligned16(prefix) || misaligned16(idx))
    return AG_ERR_INVALID_ARG;
  if (!kv_proj_cache_supported(*desc)) return AG_ERR_UNSUPPORTED;
  return launch_kv_proj_cache(*desc, X, nullptr, Wk, Wv, flags, *cache, prefix, idx, nullptr, K, V, dev_status,
                              (cudaStream_t)cuda_stream);
}

int ag_qkv_project_cache(const ag_layer_desc *desc, const void *X, const void *Wq, const void *Wk, const void *Wv,
                         const uint8_t *flags, ag_cache *cache, int32_t *prefix, int32_t *idx, void *Q, void *K,
                         void *V, int32_t *dev_status, void *cuda_stream) {
  CallRange range_("ag_qkv_project_cache");
  int st = check_desc(desc);
  if (st) return st;
  if (desc->hidden <= 0) return AG_ERR_INVALID_ARG;
  if (!X || !Wq || !Wk || !Wv || !flags || !prefix || !Q || !K || !V) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, true);
  if (st) return st;
  if (misaligned16(X) || misaligned16(Wq) || misaligned16(Wk) || misaligned16(Wv) || misaligned16(Q) ||
      misaligned16(K) || misaligned16(V) || misaligned16(flags) || misaligned16(prefix) || misaligned16(idx))
    return AG_ERR_INVALID_ARG;
  if (!kv_proj_cache_supported(*desc)) return AG_ERR_UNSUPPORTED;
  return launch_kv_proj_cache(*desc, X, Wq, Wk, Wv, flags, *cache, prefix, idx, Q, K, V, dev_status,
                              (cudaStream_t)cuda_stream);
}

int ag_prefill_attn(const ag_layer_desc *desc, const void *Q, const void *K,
                    const void *V, const uint8_t *flags, const ag_cache *cache,
                    const int32_t *prefix, float softmax_scale, void *O, void *ws,
                    size_t ws_bytes, void *cuda_stream) {
  CallRange range_("ag_prefill_attn");
  int st = check_desc(desc);
  if (st) return st;
  if (!Q || !K || !V || !flags || !prefix || !O) return AG_ERR_INVALID_ARG;
  st = check_cache(cache);
  if (st) return st;
  if (misaligned16(Q) || misaligned16(K) || misaligned16(V) || misaligned16(O) ||
      misaligned16(prefix))
    return AG_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return AG_ERR_INVALID_ARG;
  st = check_ws(prefill_workspace_bytes(*desc), ws, ws_bytes);
  if (st) return st;
  float scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)desc->head_dim) : softmax_scale;
  return launch_prefill(*desc, Q, K, V, flags, *cache, prefix, scale, O, ws,
                        (cudaStream_t)cuda_stream);
}

int ag_out_project(const ag_layer_desc *desc, const void *O, const void *Wo, const void *X_res, void *Y,
                   void *cuda_stream) {
  CallRange range_("ag_out_project");
  int st = check_desc(desc);
  if (st) return st;
  if (desc->hidden <= 0) return AG_ERR_INVALID_ARG;
  if (!O || !Wo || !Y) return AG_ERR_INVALID_ARG;
  if (misaligned16(O) || misaligned16(Wo) || misaligned16(X_res) || misaligned16(Y)) return AG_ERR_INVALID_ARG;
  if (Y == X_res || Y == O) return AG_ERR_INVALID_ARG;
  if (desc->hidden % 8 != 0) return AG_ERR_UNSUPPORTED;
  return launch_out_proj(*desc, O, Wo, X_res, Y, (cudaStream_t)cuda_stream);
}

int ag_decode_attn(const ag_layer_desc *desc, const void *q, const void *k_new,
                   const void *v_new, const ag_cache *cache, float softmax_scale,
                   void *o, void *ws, size_t ws_bytes, void *cuda_stream) {
  CallRange range_("ag_decode_attn");
  int st = check_desc(desc);
  if (st) return st;
  if (!q || !k_new || !v_new || !o) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, true);
  if (st) return st;
  if (misaligned16(q) || misaligned16(k_new) || misaligned16(v_new) || misaligned16(o))
    return AG_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return AG_ERR_INVALID_ARG;
  st = check_ws(decode_workspace_bytes(*desc), ws, ws_bytes);
  if (st) return st;
  float scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)desc->head_dim) : softmax_scale;
  return launch_decode(*desc, q, k_new, v_new, *cache, scale, o, ws, ws_bytes,
                       (cudaStream_t)cuda_stream);
}

int ag_decode_step(const ag_layer_desc *desc, const void *q, const void *k_new, const void *v_new,
                   const uint8_t *flag_new, ag_cache *cache, float softmax_scale, void *o,
                   int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream) {
  CallRange range_("ag_decode_step");
  int st = check_desc(desc);
  if (st) return st;
  if (!q || !k_new || !v_new || !flag_new || !o) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, true);
  if (st) return st;
  if (misaligned16(q) || misaligned16(k_new) || misaligned16(v_new) || misaligned16(o))
    return AG_ERR_INVALID_ARG;
  if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return AG_ERR_INVALID_ARG;
  st = check_ws(decode_workspace_bytes(*desc), ws, ws_bytes);
  if (st) return st;
  float scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)desc->head_dim) : softmax_scale;
  return launch_decode_step(*desc, q, k_new, v_new, flag_new, *cache, scale, o, dev_status, ws,
                            (cudaStream_t)cuda_stream);
}

int ag_cache_append(const ag_layer_desc *desc, const void *k_new, const void *v_new,
                    const uint8_t *flag_new, ag_cache *cache, int32_t *dev_status,
                    void *cuda_stream) {
  CallRange range_("ag_cache_append");
  int st = check_desc(desc);
  if (st) return st;
  if (!k_new || !v_new || !flag_new) return AG_ERR_INVALID_ARG;
  st = check_cache(cache, desc, true);
  if (st) return st;
  if (misaligned16(k_new) || misaligned16(v_new)) return AG_ERR_INVALID_ARG;
  return launch_append(*desc, k_new, v_new, flag_new, *cache, dev_status,
                       (cudaStream_t)cuda_stream);
}

const char *ag_status_string(int status) {
  switch (status) {
    case AG_OK: return "ok";
    case AG_ERR_INVALID_ARG: return "invalid argument";
    case AG_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case AG_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AG_ERR_CAPACITY: return "capacity exceeded";
    case AG_ERR_CUDA: return "CUDA call failed";
    default: return "unknown status";
  }
}

int ag_last_cuda_error(void) { return ag::g_last_cuda_error; }

int ag_device_wait_timeouts(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  const int a = gemm_tc_wait_timeouts(), b = prefill_tc_wait_timeouts(),
            c = gate_attn_tc_wait_timeouts() + gate_linear_wait_timeouts(), e = kv_proj_cache_wait_timeouts(),
            f = out_proj_wait_timeouts();
  return (a < 0 || b < 0 || c < 0 || e < 0 || f < 0) ? -1 : a + b + c + e + f;
}

}  // extern "C"
