/*
 * ag.h — C boundary of the Attention-Gate (AG) gated attention layer for
 * NVIDIA B200 (sm_100a).
 *
 * The layer is the inference hot path of "In-context KV-Cache Eviction for
 * LLMs via Attention-Gate" (arXiv 2410.12876):
 *
 *   ag_gate_forward   AG(X) = G(MHA'(X), tau)                 Sec. 3.3, Eq. 3, Eq. 4
 *   ag_compact_kv     keep k_i^(t), v_i^(t) iff AG(X)_i^(t)=1  Sec. 3.3 (after Eq. 4)
 *   ag_prefill_attn   Softmax(QK^T/sqrt(d_k) - INF(1-M_i))V    Eq. 2 with M_i of Eq. 5
 *   ag_decode_attn    one query over the retained cache + self Sec. 3.1 (decoding stage), Eq. 5 (j = t)
 *   ag_cache_append   concatenate the new k, v to the cache    Sec. 3.1 (decoding stage)
 *   ag_decode_step    the two above in one call                Sec. 3.1 (decoding stage)
 *   ag_gate_linear_forward  the local gate, s = X W_lin        Sec. 3.4 ("Local or global?")
 *   ag_kv_project_cache     K_i = X W^K_i, V_i = X W^V_i written
 *                           to the dense K, V and, for retained
 *                           tokens, straight into the cache     Eq. 2 + Sec. 3.3 (after Eq. 4)
 *   ag_qkv_project_cache    the same with Q_i = X W^Q_i         Eq. 2
 *   ag_out_project          [H_1 .. H_h] W^O (+ skip connection) Eq. 1
 *
 * Conventions common to every call
 * --------------------------------
 *  - Every data pointer is a DEVICE pointer unless the comment says "host".
 *    `desc` and the `ag_cache` struct itself live in HOST memory; the arrays
 *    the cache struct points to are device memory.
 *  - All tensors are dense, row-major, innermost dimension last, and every
 *    base pointer is 16-byte aligned.
 *  - Element type of X, the weights, Q, K, V, O, q, k_new, v_new, o and the
 *    cache rows is `desc->dtype` (float32 or bfloat16).  Accumulation is
 *    float32; outputs are rounded to nearest even.
 *  - Flags are one byte per (sequence, head, token): 1 = retain, 0 = evict.
 *  - The library allocates no memory and keeps no state between calls.  All
 *    buffers, the workspace and the stream belong to the caller.  Calls are
 *    asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *    the legacy default stream).
 *  - Return value: AG_OK (0) or a negative ag_status.  Argument errors are
 *    found on the host before anything is launched.  A condition only the
 *    device can see (cache slab full on append) sets a bit in a caller-owned
 *    status word and skips the write; kernels never trap.
 */
#ifndef AG_H_
#define AG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  AG_OK = 0,
  AG_ERR_INVALID_ARG = -1, /* null / misaligned pointer, non-positive size, h' >= h */
  AG_ERR_UNSUPPORTED = -2, /* shape or dtype combination without a kernel */
  AG_ERR_WORKSPACE = -3,   /* workspace missing or smaller than ag_workspace_bytes() */
  AG_ERR_CAPACITY = -4,    /* a host-known capacity bound is exceeded */
  AG_ERR_CUDA = -5         /* a CUDA runtime / driver call failed; see ag_last_cuda_error() */
} ag_status;

typedef enum { AG_F32 = 0, AG_BF16 = 1 } ag_dtype;

/* Which call a workspace query refers to. */
typedef enum {
  AG_CALL_GATE = 0,
  AG_CALL_COMPACT = 1,
  AG_CALL_PREFILL = 2,
  AG_CALL_DECODE = 3,
  AG_CALL_APPEND = 4
} ag_call;

/* Shape of one AG-gated attention layer (host memory, plain data).
 * Notation of Sec. 3.1 / 3.3: X in R^{n x d}; h heads of width d_k = d_v;
 * MHA' has h' < h heads of width d'_k and W^{O'} in R^{h' d'_k x h}. */
typedef struct {
  int32_t batch;         /* B  independent sequences                       */
  int32_t seq;           /* n  prompt length (all sequences share it)      */
  int32_t hidden;        /* d  width of X (used by ag_gate_forward only)   */
  int32_t heads;         /* h                                              */
  int32_t head_dim;      /* d_k = d_v, 64 or 128                           */
  int32_t gate_heads;    /* h' (must be < h)                               */
  int32_t gate_head_dim; /* d'_k = d'_v, 64 or 128                         */
  float tau;             /* threshold of Eq. 4, in (0, 1)                  */
  int32_t gate_causal;   /* 1: MHA' uses the lower-triangular decoder mask;
                            0: every token of MHA' sees the whole sequence  */
  int32_t dtype;         /* ag_dtype                                       */
  const int32_t *seq_lens; /* NULL, or DEVICE pointer to B lengths, 1 <= seq_lens[b] <= n:
                            sequence b is its first seq_lens[b] tokens, the rest
                            of its n positions is padding.  Read by the two gate
                            calls only: a valid token's score is what its sequence
                            alone would give (the bidirectional MHA' sees seq_lens[b]
                            keys), and every padding position gets flag 0, so it is
                            never cached and never attended to; scores and attention
                            outputs at padding positions are unspecified.  With a
                            recent-token window, ag_compact_kv and ag_kv_project_cache
                            read it too: the ring takes the last tokens of each
                            sequence's own prompt.  ag_prefill_attn skips the query
                            tiles that hold padding only.                            */
  int32_t kv_heads;      /* 0 (= heads), or the number of key/value heads of grouped-query
                            attention: heads must be a multiple; query head i reads
                            key/value head i / (heads / kv_heads).  K, V, k_new, v_new,
                            flags, flag_new, scores, prefix, idx and the cache slabs then
                            have kv_heads where the comments below say h; Q, q, O, o keep
                            h; Wo_g and W_lin have kv_heads columns.                  */
  int32_t recent_window; /* 0 or 1: the method as published, a token always sees itself and
                            otherwise only retained tokens (the diagonal of Eq. 5).
                            w in 2..17: the w most recent tokens, the current one included,
                            are visible whatever their flags (Appendix, Table 6, settings
                            (6-1), (6-2): w = 5, 10); an evicted token leaves the attention
                            of later tokens once it is w or more positions behind.  What is
                            cached for good is unchanged.  The cache then needs its
                            recent_* arrays.                                           */
} ag_layer_desc;

/* Ragged per-(sequence, head) cache of retained keys and values.  The struct
 * is host memory; every pointer in it is device memory owned by the caller.
 * Slab s = b * h + i occupies rows [row_off[s], row_off[s] + cap[s]) of both
 * row pools; its first len[s] rows are valid, in ascending token order.
 * Slabs must not overlap.  Rows of a slab beyond len[s] may hold anything. */
typedef struct {
  void *k_rows;      /* [pool_rows, head_dim] keys                          */
  void *v_rows;      /* [pool_rows, head_dim] values                        */
  int64_t pool_rows; /* rows in each pool                                   */
  int64_t *row_off;  /* [B*h] first row of each slab                        */
  int32_t *cap;      /* [B*h] rows reserved for each slab                   */
  int32_t *len;      /* [B*h] rows in use (written by compact, append)      */
  int32_t max_cap;   /* host-known upper bound of every cap[s] (sizes the
                        decode grid; must be >= max_s cap[s])               */
  /* Only with desc->recent_window = w > 1 (NULL otherwise): per slab a ring of the last
   * R = w - 1 tokens, token number p in slot p % R.  ag_compact_kv fills it from the end of
   * the prompt, ag_cache_append / ag_decode_step put every new token in (kept or not), and
   * decode attention reads the slots marked live.                                          */
  void *recent_k;       /* [B*h, R, head_dim] keys of the ring                              */
  void *recent_v;       /* [B*h, R, head_dim] values                                        */
  uint8_t *recent_live; /* [B*h, R] 1: the slot holds an EVICTED token that later tokens
                           still see (a retained one is a row of the slab already)          */
  int32_t *pos;         /* [B*h] tokens the slab has seen (prompt + appended or not)        */
} ag_cache;

/* Bits of the device status word written by ag_compact_kv / ag_cache_append. */
#define AG_DEV_OVERFLOW 1 /* a slab had no free row; the write was skipped */

/* Bytes of workspace `which` needs for this layer shape (0 = none needed).
 * Host-only; returns 0 for an invalid descriptor.  The workspace must be
 * 256-byte aligned device memory; its contents are scratch. */
size_t ag_workspace_bytes(const ag_layer_desc *desc, int which);

/*
 * Step 1 — the gate (Sec. 3.3, Eq. 3 and Eq. 4; gamma: Sec. 3.5).
 *   Q' = X Wq_g, K' = X Wk_g, V' = X Wv_g, split into h' heads of width d'_k;
 *   H'_g = Softmax(Q'_g K'_g^T / sqrt(d'_k) [causal if gate_causal]) V'_g;
 *   s = [H'_1 .. H'_h'] Wo_g                         (n x h);
 *   flag[t, i] = 1 iff Sigmoid(s[t, i] + gamma[i]) > tau   (strict).
 * The comparison is done as s + gamma > log(tau / (1 - tau)) in float32.
 *
 *   X      [B, n, d]                 in
 *   Wq_g, Wk_g, Wv_g  [d, h' d'_k]   in   ("in x out", so X W matches Eq. 2)
 *   Wo_g   [h' d'_k, h]              in
 *   gamma  [h] float32 or NULL (= 0) in
 *   scores [B, h, n] float32 or NULL out  s, head-major
 *   flags  [B, h, n] uint8           out
 */
int ag_gate_forward(const ag_layer_desc *desc, const void *X, const void *Wq_g,
                    const void *Wk_g, const void *Wv_g, const void *Wo_g,
                    const float *gamma, float *scores, uint8_t *flags, void *ws,
                    size_t ws_bytes, void *cuda_stream);

/*
 * Step 1, local variant — the gate with MHA' replaced by one linear layer
 * (Sec. 3.4, "Local or global?"; ablation setting (5)): a token's flag depends
 * on its own hidden state only.
 *   s = X W_lin                                       (n x h);
 *   flag[t, i] = 1 iff Sigmoid(s[t, i] + gamma[i]) > tau   (strict),
 * compared as s + gamma > log(tau / (1 - tau)) in float32, like ag_gate_forward.
 * Uses desc->batch, seq, hidden, heads, tau, dtype; the gate_* fields are ignored.
 * Needs no workspace.  Its flags feed ag_compact_kv and the later steps unchanged.
 *
 *   X      [B, n, d]                 in
 *   W_lin  [d, h]                    in   ("in x out")
 *   gamma  [h] float32 or NULL (= 0) in
 *   scores [B, h, n] float32 or NULL out  s, head-major
 *   flags  [B, h, n] uint8           out
 * Returns AG_ERR_INVALID_ARG for missing or misaligned (16-byte) pointers or a
 * tau outside (0, 1); AG_ERR_CUDA if a launch fails.
 */
int ag_gate_linear_forward(const ag_layer_desc *desc, const void *X, const void *W_lin,
                           const float *gamma, float *scores, uint8_t *flags,
                           void *cuda_stream);

/*
 * Step 2 — selective caching (Sec. 3.3: k_i^(t), v_i^(t) are retained iff
 * AG(X)_i^(t) = 1).  For every slab s = (b, i):
 *   prefix[s, j] = #{t < j : flags[s, t] = 1}, j = 0..n  (prefix[s, n] = L_s);
 *   idx[s, r]    = r-th retained position (ascending), r < L_s;
 *   cache rows row_off[s] + r  <-  K[s, idx[s, r]], V[s, idx[s, r]] (bit copies);
 *   cache.len[s] = L_s.
 * If L_s > cap[s] nothing is copied for that slab, len[s] is set to 0 and
 * AG_DEV_OVERFLOW is or-ed into *dev_status.
 * With K = V = NULL only prefix, idx and len are produced (a count pass that
 * lets the caller lay out tight slabs before the copying pass).
 *
 *   K, V    [B, h, n, D]          in (or both NULL)
 *   flags   [B, h, n] uint8       in
 *   cache   host struct           in/out (len; k_rows, v_rows)
 *   prefix  [B, h, n + 1] int32   out
 *   idx     [B, h, n] int32 or NULL  out (entries r >= L_s are left untouched)
 *   dev_status  int32 or NULL     in/out (bits are or-ed in)
 */
int ag_compact_kv(const ag_layer_desc *desc, const void *K, const void *V,
                  const uint8_t *flags, ag_cache *cache, int32_t *prefix,
                  int32_t *idx, int32_t *dev_status, void *ws, size_t ws_bytes,
                  void *cuda_stream);

/*
 * Step 2 fused with the projection that feeds it — the key/value projection of Eq. 2,
 *   K_i = X W^K_i,  V_i = X W^V_i      (head i = columns [i D, (i + 1) D) of the weight),
 * and selective caching (Sec. 3.3: k_i^(t), v_i^(t) are retained iff
 * AG(X)_i^(t) = 1) in one call.  Each projected tile is rounded to the layer
 * dtype once and written to both places the layer reads it from: the dense K, V
 * (every token attends to its own key and value, the diagonal of Eq. 5) and,
 * for retained tokens, cache row row_off[s] + prefix[s, t].  prefix, idx and
 * len are computed from the flags as ag_compact_kv computes them.  A layer that
 * owns its key/value projection calls gate -> this call -> ag_prefill_attn, and
 * ag_compact_kv not at all.
 *
 *   X       [B, n, d]             in
 *   Wk, Wv  [d, h D]              in   ("in x out")
 *   flags   [B, h, n] uint8       in
 *   cache   host struct           in/out: k_rows, v_rows of the retained tokens, len[s] = L_s
 *   prefix  [B, h, n + 1] int32   out  exclusive counts of the flags, prefix[s, n] = L_s
 *   idx     [B, h, n] int32 or NULL  out  (entries r >= L_s are left untouched)
 *   K, V    [B, h, n, D]          out  dense projections (h = kv_heads for grouped-query attention)
 *   dev_status  int32 or NULL     in/out
 * A slab with L_s > cap[s] gets no rows, len[s] = 0 and AG_DEV_OVERFLOW, as in
 * ag_compact_kv.  The cache rows are bit copies of the dense K, V rows.
 * With a recent-token window the ring of the cache is filled from the dense K, V,
 * as ag_compact_kv fills it.
 * Needs no workspace.  Kernel coverage: bfloat16, head_dim 128, d a multiple of 8
 * (any batch, any n); anything else returns AG_ERR_UNSUPPORTED (project with a
 * GEMM of your own and call ag_compact_kv).
 * AG_ERR_INVALID_ARG for missing or misaligned (16-byte) pointers.
 */
int ag_kv_project_cache(const ag_layer_desc *desc, const void *X, const void *Wk,
                        const void *Wv, const uint8_t *flags, ag_cache *cache,
                        int32_t *prefix, int32_t *idx, void *K, void *V,
                        int32_t *dev_status, void *cuda_stream);

/*
 * ag_kv_project_cache with the query projection of Eq. 2, Q_i = X W^Q_i, in the
 * same launch: the whole Q, K, V projection of the layer runs inside the path.
 * Queries take no part in eviction: Q goes to its dense tensor only.
 *
 *   Wq      [d, heads D]          in   ("in x out")
 *   Q       [B, heads, n, D]      out
 * Everything else (arguments, results, kernel coverage, errors) as for
 * ag_kv_project_cache; with grouped-query attention Q has desc->heads heads and
 * K, V, flags, prefix, idx and the cache desc->kv_heads.
 */
int ag_qkv_project_cache(const ag_layer_desc *desc, const void *X, const void *Wq,
                         const void *Wk, const void *Wv, const uint8_t *flags,
                         ag_cache *cache, int32_t *prefix, int32_t *idx, void *Q,
                         void *K, void *V, int32_t *dev_status, void *cuda_stream);

/*
 * Step 3 — prefill attention under the eviction mask (Eq. 2 with Eq. 5):
 *   O_i[j] = sum_t A_i[j, t] V_i[t],
 *   A_i = row-Softmax(Q_i K_i^T * scale - INF (1 - M_i)),
 *   M_i[j, t] = 1 if t = j;  flags_i[t] if t < j;  0 if t > j.
 * The kernel reads the retained keys from the compacted cache (rows
 * r < prefix[s, j] are exactly the retained t < j) and the self term from
 * the dense K, V, so `cache` and `prefix` must be those ag_compact_kv wrote
 * for the same K, V, flags.
 *
 *   Q, K, V [B, h, n, D]  in      softmax_scale: 0 means 1/sqrt(D)
 *   O       [B, h, n, D]  out
 */
int ag_prefill_attn(const ag_layer_desc *desc, const void *Q, const void *K,
                    const void *V, const uint8_t *flags, const ag_cache *cache,
                    const int32_t *prefix, float softmax_scale, void *O,
                    void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Downstream of step 3 — the layer's output, Eq. 1: MHA(X) = [H_1(X), ..., H_h(X)] W^O, the
 * heads' outputs concatenated along the feature axis (head i in columns [i D, (i + 1) D)) and
 * projected by W^O in R^{h D x d}; with X_res, the Transformer's skip connection is added in the
 * same pass:
 *   Y[b, t, :] = X_res[b, t, :] + sum_i O[b, i, t, :] Wo[i D : (i + 1) D, :].
 * The paper stops at Eq. 1; the skip connection is what feeds a layer's output to the next layer
 * in a stack of attention layers (no normalisation, no feed-forward block in between).
 * Float32 accumulation, one rounding to the layer dtype.  Uses desc->batch, seq, heads, head_dim,
 * hidden, dtype.  Needs no workspace.
 *
 *   O      [B, h, n, D]          in   (as ag_prefill_attn writes it; h = desc->heads)
 *   Wo     [h D, d]              in   ("in x out")
 *   X_res  [B, n, d] or NULL     in   skip connection (NULL: Y = MHA(X))
 *   Y      [B, n, d]             out  must not be X_res or O
 * Tensor-core coverage: bfloat16, head_dim 128, d a multiple of 128; other shapes run on
 * CUDA cores (B n <= 65535), else AG_ERR_UNSUPPORTED.
 * AG_ERR_INVALID_ARG for missing or misaligned (16-byte) pointers.
 */
int ag_out_project(const ag_layer_desc *desc, const void *O, const void *Wo, const void *X_res,
                   void *Y, void *cuda_stream);

/*
 * Step 4a — one decode query per (sequence, head) (Sec. 3.1 decoding stage;
 * the cache holds only retained tokens, Sec. 3.3; the token always sees its
 * own key, Eq. 5 case j = t):
 *   o[s] = Softmax([q[s] . Kc_s^T, q[s] . k_new[s]] * scale) [Vc_s; v_new[s]]
 * over the len[s] valid rows of slab s.  len[s] = 0 gives o[s] = v_new[s].
 * Does not modify the cache.
 *
 *   q, k_new, v_new [B, h, D]  in      o [B, h, D]  out
 */
int ag_decode_attn(const ag_layer_desc *desc, const void *q, const void *k_new,
                   const void *v_new, const ag_cache *cache,
                   float softmax_scale, void *o, void *ws, size_t ws_bytes,
                   void *cuda_stream);

/*
 * Step 4b — conditional append (Sec. 3.1: the new k, v are concatenated to
 * the cache; here only when the token's flag retains it):
 *   if flag_new[s]: rows row_off[s] + len[s] <- k_new[s], v_new[s]; len[s] += 1.
 * A full slab (len[s] = cap[s]) skips the write and or-s AG_DEV_OVERFLOW into
 * *dev_status.
 *
 *   k_new, v_new [B, h, D]   in      flag_new [B, h] uint8  in
 *   dev_status   int32 or NULL  in/out
 */
int ag_cache_append(const ag_layer_desc *desc, const void *k_new,
                    const void *v_new, const uint8_t *flag_new, ag_cache *cache,
                    int32_t *dev_status, void *cuda_stream);

/*
 * Steps 4a + 4b in one call (Sec. 3.1, decoding stage): the attention of
 * ag_decode_attn over the cache as it stands, then the conditional append of
 * ag_cache_append, carried by the same kernels (the slab's rows and length are
 * read before the new row goes in, so o is exactly what ag_decode_attn gives
 * and the cache ends exactly as ag_cache_append leaves it).  One decode step
 * of a layer is one such call; it saves a launch per step.
 *
 *   q, k_new, v_new [B, h, D]  in      flag_new [B, h] uint8  in
 *   o [B, h, D]  out                   dev_status int32 or NULL  in/out
 * Workspace and errors as for ag_decode_attn (AG_CALL_DECODE).
 */
int ag_decode_step(const ag_layer_desc *desc, const void *q, const void *k_new,
                   const void *v_new, const uint8_t *flag_new, ag_cache *cache,
                   float softmax_scale, void *o, int32_t *dev_status, void *ws,
                   size_t ws_bytes, void *cuda_stream);

/*
 * ag_decode_attn without any caller-supplied scratch.  The paper has no
 * counterpart to this call; it exists for integration reasons only.
 *
 * Who needs it: code that runs where device memory cannot be requested —
 * for example a plug-in inside a serving process that handed the whole GPU
 * to its own memory pool at start-up (a later cudaMalloc simply fails), or a
 * latency-critical step that must not hit the device-wide synchronisation an
 * allocation can cause.  Such a caller has pointers to its inputs and outputs
 * and nothing else, so it cannot provide the split-K workspace that
 * ag_decode_attn asks for.
 *
 * This variant computes exactly what ag_decode_attn computes, with the
 * workspace replaced by a fixed 17,039,360-byte array that is part of the
 * library image (every GPU that loads the library holds it until the process
 * exits).  It calls no allocation routine of any kind.  (Up to 64 slabs
 * neither the workspace nor the array is touched: that form of the kernel
 * keeps its partial results on chip.)
 *
 *  - Limit: batch * heads * 32 * (head_dim + 2) * 4 bytes must fit in the
 *    array, i.e. batch * heads <= 1024 at head_dim 128 (2016 at head_dim 64).
 *    Larger problems are refused with AG_ERR_CAPACITY before any launch.
 *  - The first call on each device looks up the array's device address (the
 *    device must be current, as for every call).  Make that first call
 *    outside any stream capture.
 *  - A layer with desc->recent_window > 1 is refused with AG_ERR_UNSUPPORTED:
 *    this entry does not read the ring of recent tokens.
 *  - All calls share the one array.  Its previous contents never matter (each
 *    call writes every partial result before reading it), but two calls that
 *    may overlap on the GPU — different streams, or different host threads
 *    on the same device — race on it.  Serialise them, or use ag_decode_attn
 *    with separate workspaces.
 *
 * Arguments, layouts and return values are those of ag_decode_attn.
 */
int ag_decode_attn_noalloc(const ag_layer_desc *desc, const void *q,
                           const void *k_new, const void *v_new,
                           const ag_cache *cache, float softmax_scale, void *o,
                           void *cuda_stream);

/* Text for an ag_status (static storage, never NULL). */
const char *ag_status_string(int status);

/* cudaError_t value of the most recent failed CUDA call made by this library
 * on the calling thread (0 if none). */
int ag_last_cuda_error(void);

/* Diagnostic: number of bounded device-side waits (on a TMA load or a tensor-core
 * completion) that expired in this library's kernels on the current device since
 * the library was loaded.  0 in a healthy run; a kernel whose wait expired
 * unwound cleanly but its output is not valid.  Returns -1 if the counter
 * cannot be read.  Synchronises the device. */
int ag_device_wait_timeouts(void);

#ifdef __cplusplus
}
#endif
#endif /* AG_H_ */
