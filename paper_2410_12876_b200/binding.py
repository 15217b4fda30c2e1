"""ctypes binding of libag.so: argument marshalling only.

Each function has the name and argument order of its C counterpart in
include/ag.h and does nothing but turn torch tensors into device pointers.
Every step of the layer runs inside the CUDA library; there is no Python or
CPU fallback, and loading fails loudly when the library has not been built.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libag.so")

AG_F32, AG_BF16 = 0, 1
AG_CALL_GATE, AG_CALL_COMPACT, AG_CALL_PREFILL, AG_CALL_DECODE, AG_CALL_APPEND = range(5)
AG_OK, AG_ERR_INVALID_ARG, AG_ERR_UNSUPPORTED, AG_ERR_WORKSPACE, AG_ERR_CAPACITY, AG_ERR_CUDA = 0, -1, -2, -3, -4, -5
AG_DEV_OVERFLOW = 1

EXPORTS = (
    "ag_workspace_bytes", "ag_gate_forward", "ag_compact_kv", "ag_prefill_attn",
    "ag_decode_attn", "ag_cache_append", "ag_status_string", "ag_last_cuda_error",
    "ag_decode_attn_noalloc", "ag_device_wait_timeouts", "ag_gate_linear_forward", "ag_decode_step",
    "ag_kv_project_cache", "ag_qkv_project_cache", "ag_out_project",
)


class AgError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {ag_status_string(status)} ({status})")


class ag_layer_desc(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("hidden", ctypes.c_int32),
        ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("gate_heads", ctypes.c_int32), ("gate_head_dim", ctypes.c_int32),
        ("tau", ctypes.c_float), ("gate_causal", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("seq_lens", ctypes.c_void_p), ("kv_heads", ctypes.c_int32), ("recent_window", ctypes.c_int32),
    ]


class ag_cache(ctypes.Structure):
    _fields_ = [
        ("k_rows", ctypes.c_void_p), ("v_rows", ctypes.c_void_p), ("pool_rows", ctypes.c_int64),
        ("row_off", ctypes.c_void_p), ("cap", ctypes.c_void_p), ("len", ctypes.c_void_p),
        ("max_cap", ctypes.c_int32),
        ("recent_k", ctypes.c_void_p), ("recent_v", ctypes.c_void_p), ("recent_live", ctypes.c_void_p),
        ("pos", ctypes.c_void_p),
    ]


_lib = None


def lib():
    """The loaded CUDA library; raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2410_12876_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        dp, cp = ctypes.POINTER(ag_layer_desc), ctypes.POINTER(ag_cache)
        L.ag_workspace_bytes.restype = sz
        L.ag_workspace_bytes.argtypes = [dp, i32]
        L.ag_gate_forward.restype = i32
        L.ag_gate_forward.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.ag_gate_linear_forward.restype = i32
        L.ag_gate_linear_forward.argtypes = [dp, vp, vp, vp, vp, vp, vp]
        L.ag_compact_kv.restype = i32
        L.ag_compact_kv.argtypes = [dp, vp, vp, vp, cp, vp, vp, vp, vp, sz, vp]
        L.ag_kv_project_cache.restype = i32
        L.ag_kv_project_cache.argtypes = [dp, vp, vp, vp, vp, cp, vp, vp, vp, vp, vp, vp]
        L.ag_qkv_project_cache.restype = i32
        L.ag_qkv_project_cache.argtypes = [dp, vp, vp, vp, vp, vp, cp, vp, vp, vp, vp, vp, vp, vp]
        L.ag_out_project.restype = i32
        L.ag_out_project.argtypes = [dp, vp, vp, vp, vp, vp]
        L.ag_prefill_attn.restype = i32
        L.ag_prefill_attn.argtypes = [dp, vp, vp, vp, vp, cp, vp, f32, vp, vp, sz, vp]
        L.ag_decode_attn.restype = i32
        L.ag_decode_attn.argtypes = [dp, vp, vp, vp, cp, f32, vp, vp, sz, vp]
        L.ag_decode_step.restype = i32
        L.ag_decode_step.argtypes = [dp, vp, vp, vp, vp, cp, f32, vp, vp, vp, sz, vp]
        L.ag_decode_attn_noalloc.restype = i32
        L.ag_decode_attn_noalloc.argtypes = [dp, vp, vp, vp, cp, f32, vp, vp]
        L.ag_cache_append.restype = i32
        L.ag_cache_append.argtypes = [dp, vp, vp, vp, cp, vp, vp]
        L.ag_status_string.restype = ctypes.c_char_p
        L.ag_status_string.argtypes = [i32]
        L.ag_last_cuda_error.restype = i32
        L.ag_last_cuda_error.argtypes = []
        L.ag_device_wait_timeouts.restype = i32
        L.ag_device_wait_timeouts.argtypes = []
        _lib = L
    return _lib


def make_desc(shape, seq_lens=None):
    """ag_layer_desc from an object with the LayerShape fields; seq_lens: optional int32 device
    tensor [batch] of sequence lengths (the caller keeps it alive while the descriptor is used)."""
    if seq_lens is not None:
        assert seq_lens.dtype == torch.int32 and seq_lens.is_cuda and seq_lens.numel() == shape.batch
    return ag_layer_desc(shape.batch, shape.seq, shape.hidden, shape.heads, shape.head_dim,
                         shape.gate_heads, shape.gate_head_dim, float(shape.tau),
                         int(shape.gate_causal), AG_F32 if shape.dtype == "f32" else AG_BF16,
                         None if seq_lens is None else seq_lens.data_ptr(), int(getattr(shape, "kv_heads", 0)),
                         int(getattr(shape, "recent_window", 0)))


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _ws(ws):
    if ws is None:
        return None, 0
    return ws.data_ptr(), ws.numel() * ws.element_size()


class RaggedCache:
    """Device buffers of a ragged retained-KV cache plus the host struct the
    C calls take.  Holds references so the tensors outlive the struct."""

    def __init__(self, k_rows, v_rows, row_off, cap, length, max_cap, recent=None):
        self.k_rows, self.v_rows, self.row_off, self.cap, self.len = k_rows, v_rows, row_off, cap, length
        self.max_cap = int(max_cap)
        # ring of the last recent_window - 1 tokens of every slab: (keys, values, live marks, tokens seen)
        self.recent_k, self.recent_v, self.recent_live, self.pos = recent if recent is not None else (None,) * 4
        self.struct = ag_cache(_ptr(k_rows), _ptr(v_rows), int(k_rows.shape[0]), _ptr(row_off),
                               _ptr(cap), _ptr(length), self.max_cap, _ptr(self.recent_k), _ptr(self.recent_v),
                               _ptr(self.recent_live), _ptr(self.pos))

    @classmethod
    def allocate(cls, shape, cap, device="cuda"):
        """Back-to-back slabs with the given per-slab capacities (int array [B*h])."""
        import numpy as np
        cap = np.asarray(cap, dtype=np.int64)
        off = np.zeros(cap.size, dtype=np.int64)
        off[1:] = np.cumsum(cap[:-1])
        pool = int(cap.sum())
        k = torch.zeros(max(pool, 1), shape.head_dim, dtype=shape.torch_dtype, device=device)
        v = torch.zeros_like(k)
        recent = None
        R = int(getattr(shape, "recent_window", 0)) - 1
        if R > 0:
            rk = torch.zeros(cap.size, R, shape.head_dim, dtype=shape.torch_dtype, device=device)
            recent = (rk, torch.zeros_like(rk), torch.zeros(cap.size, R, dtype=torch.uint8, device=device),
                      torch.zeros(cap.size, dtype=torch.int32, device=device))
        return cls(k[:pool], v[:pool],
                   torch.from_numpy(off).to(device),
                   torch.from_numpy(cap.astype("int32")).to(device),
                   torch.zeros(cap.size, dtype=torch.int32, device=device),
                   int(cap.max()) if cap.size else 0, recent)


def ag_status_string(status):
    return lib().ag_status_string(int(status)).decode()


def ag_last_cuda_error():
    return lib().ag_last_cuda_error()


def ag_device_wait_timeouts():
    return lib().ag_device_wait_timeouts()


def ag_workspace_bytes(desc, which):
    return int(lib().ag_workspace_bytes(ctypes.byref(desc), int(which)))


def _check(st, where):
    if st != AG_OK:
        raise AgError(st, where)
    return st


def ag_gate_forward(desc, X, Wq_g, Wk_g, Wv_g, Wo_g, gamma, scores, flags, ws, stream=None):
    p, nbytes = _ws(ws)
    return _check(lib().ag_gate_forward(ctypes.byref(desc), _ptr(X), _ptr(Wq_g), _ptr(Wk_g), _ptr(Wv_g),
                                        _ptr(Wo_g), _ptr(gamma), _ptr(scores), _ptr(flags), p, nbytes,
                                        _stream(stream)), "ag_gate_forward")


def ag_gate_linear_forward(desc, X, W_lin, gamma, scores, flags, stream=None):
    return _check(lib().ag_gate_linear_forward(ctypes.byref(desc), _ptr(X), _ptr(W_lin), _ptr(gamma), _ptr(scores),
                                               _ptr(flags), _stream(stream)), "ag_gate_linear_forward")


def ag_compact_kv(desc, K, V, flags, cache, prefix, idx, dev_status, ws, stream=None):
    p, nbytes = _ws(ws)
    return _check(lib().ag_compact_kv(ctypes.byref(desc), _ptr(K), _ptr(V), _ptr(flags),
                                      ctypes.byref(cache.struct), _ptr(prefix), _ptr(idx),
                                      _ptr(dev_status), p, nbytes, _stream(stream)), "ag_compact_kv")


def ag_kv_project_cache(desc, X, Wk, Wv, flags, cache, prefix, idx, K, V, dev_status, stream=None):
    return _check(lib().ag_kv_project_cache(ctypes.byref(desc), _ptr(X), _ptr(Wk), _ptr(Wv), _ptr(flags),
                                            ctypes.byref(cache.struct), _ptr(prefix), _ptr(idx), _ptr(K), _ptr(V),
                                            _ptr(dev_status), _stream(stream)), "ag_kv_project_cache")


def ag_qkv_project_cache(desc, X, Wq, Wk, Wv, flags, cache, prefix, idx, Q, K, V, dev_status, stream=None):
    return _check(lib().ag_qkv_project_cache(ctypes.byref(desc), _ptr(X), _ptr(Wq), _ptr(Wk), _ptr(Wv), _ptr(flags),
                                             ctypes.byref(cache.struct), _ptr(prefix), _ptr(idx), _ptr(Q), _ptr(K),
                                             _ptr(V), _ptr(dev_status), _stream(stream)), "ag_qkv_project_cache")


def ag_prefill_attn(desc, Q, K, V, flags, cache, prefix, softmax_scale, O, ws, stream=None):
    p, nbytes = _ws(ws)
    return _check(lib().ag_prefill_attn(ctypes.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _ptr(flags),
                                        ctypes.byref(cache.struct), _ptr(prefix), float(softmax_scale),
                                        _ptr(O), p, nbytes, _stream(stream)), "ag_prefill_attn")


def ag_out_project(desc, O, Wo, X_res, Y, stream=None):
    return _check(lib().ag_out_project(ctypes.byref(desc), _ptr(O), _ptr(Wo), _ptr(X_res), _ptr(Y), _stream(stream)),
                  "ag_out_project")


def ag_decode_attn(desc, q, k_new, v_new, cache, softmax_scale, o, ws, stream=None):
    p, nbytes = _ws(ws)
    return _check(lib().ag_decode_attn(ctypes.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new),
                                       ctypes.byref(cache.struct), float(softmax_scale), _ptr(o), p, nbytes,
                                       _stream(stream)), "ag_decode_attn")


def ag_decode_attn_noalloc(desc, q, k_new, v_new, cache, softmax_scale, o, stream=None):
    """ag_decode_attn for callers that have no device memory to offer as
    workspace (see include/ag.h): same result, scratch held inside the library,
    no allocation.  Calls on one device must not overlap; batch * heads is
    limited (1024 at head_dim 128), beyond which AgError(AG_ERR_CAPACITY)."""
    return _check(lib().ag_decode_attn_noalloc(ctypes.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new),
                                               ctypes.byref(cache.struct), float(softmax_scale), _ptr(o),
                                               _stream(stream)), "ag_decode_attn_noalloc")


def ag_decode_step(desc, q, k_new, v_new, flag_new, cache, softmax_scale, o, dev_status, ws, stream=None):
    p, nbytes = _ws(ws)
    return _check(lib().ag_decode_step(ctypes.byref(desc), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(flag_new),
                                       ctypes.byref(cache.struct), float(softmax_scale), _ptr(o), _ptr(dev_status),
                                       p, nbytes, _stream(stream)), "ag_decode_step")


def ag_cache_append(desc, k_new, v_new, flag_new, cache, dev_status, stream=None):
    return _check(lib().ag_cache_append(ctypes.byref(desc), _ptr(k_new), _ptr(v_new), _ptr(flag_new),
                                        ctypes.byref(cache.struct), _ptr(dev_status), _stream(stream)),
                  "ag_cache_append")


def workspace(desc, which, device="cuda"):
    """A device buffer of ag_workspace_bytes(desc, which) bytes (None if 0)."""
    n = ag_workspace_bytes(desc, which)
    if n == 0:
        return None
    return torch.empty(n, dtype=torch.uint8, device=device)
