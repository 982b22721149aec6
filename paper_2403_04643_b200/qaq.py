"""ctypes binding of libqaq.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the
library's CUDA kernels.  Loading fails loudly when the library has not been built --
there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libqaq.so")
_lib = None

QAQ_OK = 0
TILE_TOKENS = 64
EXPORTED = [
    "qaq_status_string", "qaq_last_cuda_error", "qaq_cache_create", "qaq_cache_destroy", "qaq_cache_reset", "qaq_cache_tokens",
    "qaq_policy_from_hyper", "qaq_thresholds_workspace_bytes", "qaq_outlier_thresholds", "qaq_select_bits",
    "qaq_quantize_append", "qaq_decode_workspace_bytes", "qaq_decode_attention", "qaq_quantize_append_host",
    "qaq_decode_attention_host", "qaq_cache_stats", "qaq_cache_export", "qaq_decode_attention_static",
    "qaq_requantize_down", "qaq_requantize", "qaq_cache_compact", "qaq_cache_pool_use", "qaq_prefill_window_workspace_bytes", "qaq_prefill_window",
    "qaq_qnorm2_quantile", "qaq_decode_multi_workspace_bytes", "qaq_decode_attention_multi",
    "qaq_stream_begin", "qaq_stream_append", "qaq_stream_decode", "qaq_stream_end",
]


class QaqError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        detail = f" [{lib().qaq_last_cuda_error().decode()}]" if int(code) == 4 else ""
        super().__init__(f"{where}: {status_string(code)} ({int(code)}){detail}")


class Config(C.Structure):
    _fields_ = [("batch", C.c_int), ("heads", C.c_int), ("head_dim", C.c_int), ("max_tokens", C.c_int),
                ("bits_min", C.c_int), ("bits_max", C.c_int), ("window", C.c_int), ("outlier_frac", C.c_double),
                ("max_outliers_per_bh", C.c_long)]


class Policy(C.Structure):
    _fields_ = [("cK", C.c_float), ("cV", C.c_float)]


class Stats(C.Structure):
    _fields_ = [("tokens", C.c_long), ("code_bytes", C.c_long * 2), ("outliers", C.c_long * 2),
                ("hist", (C.c_long * 9) * 2), ("resident_bytes", C.c_long), ("cr_paper", C.c_double),
                ("cr_total", C.c_double), ("device_status", C.c_int)]


def lib():
    """The loaded library; raises if libqaq.so is missing (build it with paper_2403_04643_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} not found: run `python -m paper_2403_04643_b200.build` first "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(_LIB_PATH)
        L.qaq_status_string.restype = C.c_char_p
        L.qaq_last_cuda_error.restype = C.c_char_p
        L.qaq_last_cuda_error.argtypes = []
        L.qaq_status_string.argtypes = [C.c_int]
        L.qaq_cache_tokens.restype = C.c_long
        L.qaq_cache_tokens.argtypes = [C.c_void_p]
        L.qaq_cache_create.argtypes = [C.POINTER(Config), C.POINTER(C.c_void_p)]
        L.qaq_cache_destroy.argtypes = [C.c_void_p]
        L.qaq_cache_reset.argtypes = [C.c_void_p, C.c_void_p]
        L.qaq_policy_from_hyper.argtypes = [C.c_double, C.c_double, C.c_double, C.c_long, C.POINTER(Policy)]
        L.qaq_thresholds_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
        L.qaq_outlier_thresholds.argtypes = [C.POINTER(Config), C.c_void_p, C.c_void_p, C.c_long, C.c_long, C.c_long,
                                             C.c_int, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qaq_select_bits.argtypes = [C.POINTER(Config), C.POINTER(Policy), C.c_void_p, C.c_void_p, C.c_long, C.c_long,
                                      C.c_long, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p]
        L.qaq_quantize_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_long, C.c_long, C.c_long, C.c_int,
                                          C.c_void_p, C.c_void_p, C.POINTER(Policy), C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p]
        L.qaq_decode_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        L.qaq_decode_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_size_t, C.c_void_p]
        L.qaq_quantize_append_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.POINTER(Policy),
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.qaq_decode_attention_host.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]
        L.qaq_decode_attention_static.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]
        L.qaq_cache_stats.argtypes = [C.c_void_p, C.POINTER(Stats), C.c_void_p]
        L.qaq_prefill_window_workspace_bytes.argtypes = [C.POINTER(Config), C.c_int, C.POINTER(C.c_size_t)]
        L.qaq_prefill_window.argtypes = [C.POINTER(Config), C.c_void_p, C.c_void_p, C.c_long, C.c_long, C.c_long, C.c_int,
                                         C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qaq_qnorm2_quantile.argtypes = [C.c_void_p, C.c_long, C.c_double, C.c_void_p, C.c_void_p]
        L.qaq_decode_multi_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
        L.qaq_decode_attention_multi.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qaq_stream_begin.argtypes = [C.c_void_p, C.c_void_p]
        L.qaq_stream_end.argtypes = [C.c_void_p, C.c_void_p]
        L.qaq_stream_append.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_long, C.c_long, C.c_void_p, C.c_void_p,
                                        C.POINTER(Policy), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.qaq_stream_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_long, C.c_void_p,
                                        C.c_size_t, C.c_void_p]
        L.qaq_cache_compact.argtypes = [C.c_void_p, C.c_void_p]
        L.qaq_cache_pool_use.argtypes = [C.c_void_p, C.POINTER(C.c_long), C.POINTER(C.c_long), C.c_void_p]
        L.qaq_requantize.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_long, C.c_long, C.c_long, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.POINTER(Policy), C.c_void_p, C.c_void_p, C.c_long, C.c_void_p]
        L.qaq_requantize_down.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(Policy), C.c_void_p, C.c_void_p,
                                          C.c_long, C.c_void_p]
        L.qaq_cache_export.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_long, C.c_void_p, C.c_void_p, C.c_void_p, C.c_long, C.c_void_p]
        _lib = L
    return _lib


def status_string(code) -> str:
    return lib().qaq_status_string(int(code)).decode()


def _check(code, where):
    if code != QAQ_OK:
        raise QaqError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _strides(x):
    assert x.dim() == 4 and x.stride(3) == 1 and x.dtype == torch.float16
    return x.stride(0), x.stride(1), x.stride(2)


def make_config(batch, heads, head_dim, max_tokens, bits_min=2, bits_max=8, window=1, outlier_frac=0.01,
                max_outliers_per_bh=0) -> Config:
    return Config(batch, heads, head_dim, max_tokens, bits_min, bits_max, window, outlier_frac, max_outliers_per_bh)


def qaq_policy_from_hyper(sigmaS_max, sigmaX_max, qnorm2, T) -> Policy:
    p = Policy()
    _check(lib().qaq_policy_from_hyper(sigmaS_max, sigmaX_max, qnorm2, T, C.byref(p)), "qaq_policy_from_hyper")
    return p


class Cache:
    """Owner of a qaq_cache handle."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self._h = C.c_void_p()
        _check(lib().qaq_cache_create(C.byref(cfg), C.byref(self._h)), "qaq_cache_create")
        n = C.c_size_t()
        _check(lib().qaq_decode_workspace_bytes(self._h, C.byref(n)), "qaq_decode_workspace_bytes")
        self.decode_ws_bytes = n.value
        self._ws = None

    @property
    def handle(self):
        return self._h

    @property
    def tokens(self) -> int:
        return int(lib().qaq_cache_tokens(self._h))

    def workspace(self):
        if self._ws is None:
            self._ws = torch.empty(self.decode_ws_bytes, dtype=torch.uint8, device="cuda")
        return self._ws

    def reset(self):
        _check(lib().qaq_cache_reset(self._h, _stream()), "qaq_cache_reset")

    def close(self):
        if self._h:
            lib().qaq_cache_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def qaq_outlier_thresholds(cfg: Config, K, V, thr=None):
    sb, sh, st = _strides(K)
    assert _strides(V) == (sb, sh, st)
    BH = cfg.batch * cfg.heads
    if thr is None:
        thr = torch.empty((BH, 4), dtype=torch.float32, device=K.device)
    n = C.c_size_t()
    _check(lib().qaq_thresholds_workspace_bytes(C.byref(cfg), C.byref(n)), "qaq_thresholds_workspace_bytes")
    ws = torch.empty(n.value, dtype=torch.uint8, device=K.device)
    _check(lib().qaq_outlier_thresholds(C.byref(cfg), _ptr(K), _ptr(V), sb, sh, st, K.shape[2], _ptr(thr), _ptr(ws),
                                        n.value, _stream()), "qaq_outlier_thresholds")
    return thr


def qaq_select_bits(cfg: Config, policy: Policy, K, V, ring, nvalid, thr):
    sb, sh, st = _strides(K)
    BH, n = cfg.batch * cfg.heads, K.shape[2]
    bitsK = torch.empty((BH, n), dtype=torch.uint8, device=K.device)
    bitsV = torch.empty((BH, n), dtype=torch.uint8, device=K.device)
    _check(lib().qaq_select_bits(C.byref(cfg), C.byref(policy), _ptr(K), _ptr(V), sb, sh, st, n, _ptr(ring), _ptr(nvalid),
                                 _ptr(thr), _ptr(bitsK), _ptr(bitsV), _stream()), "qaq_select_bits")
    return bitsK, bitsV


def qaq_quantize_append(cache: Cache, K_new, V_new, thr, *, bitsK=None, bitsV=None, policy=None, ring=None, nvalid=None):
    sb, sh, st = _strides(K_new)
    assert _strides(V_new) == (sb, sh, st)
    pol = C.byref(policy) if policy is not None else None
    _check(lib().qaq_quantize_append(cache.handle, _ptr(K_new), _ptr(V_new), sb, sh, st, K_new.shape[2], _ptr(bitsK),
                                     _ptr(bitsV), pol, _ptr(ring), _ptr(nvalid), _ptr(thr), _stream()),
           "qaq_quantize_append")


def qaq_prefill_window(cfg: Config, Q, K, softmax_scale, want_qnorm2=False):
    """Score window after a prefill: Q [B*H, window, D] (the last `window` queries), K [B,H,T,D], both fp16 on the
    device.  Returns (ring [B,H,window,T] fp32, nvalid [B,H,T] u8[, qnorm2 [B*H, window]])."""
    sb, sh, st = _strides(K)
    BH, T, n = cfg.batch * cfg.heads, K.shape[2], cfg.window
    assert Q.dtype == torch.float16 and Q.is_contiguous() and Q.numel() == BH * n * cfg.head_dim
    ring = torch.empty((cfg.batch, cfg.heads, n, T), dtype=torch.float32, device=K.device)
    nvalid = torch.empty((cfg.batch, cfg.heads, T), dtype=torch.uint8, device=K.device)
    qn = torch.empty((BH, n), dtype=torch.float32, device=K.device) if want_qnorm2 else None
    nb = C.c_size_t()
    _check(lib().qaq_prefill_window_workspace_bytes(C.byref(cfg), T, C.byref(nb)), "qaq_prefill_window_workspace_bytes")
    ws = torch.empty(max(nb.value, 8), dtype=torch.uint8, device=K.device)
    _check(lib().qaq_prefill_window(C.byref(cfg), _ptr(Q), _ptr(K), sb, sh, st, T, float(softmax_scale), _ptr(ring),
                                    _ptr(nvalid), _ptr(qn), _ptr(ws), ws.numel(), _stream()), "qaq_prefill_window")
    return (ring, nvalid, qn) if want_qnorm2 else (ring, nvalid)


def qaq_qnorm2_quantile(values, upper_frac=0.1, out=None):
    """Upper quantile of squared query norms (fp32 tensor on the device, any shape); returns a 1-element device tensor."""
    assert values.dtype == torch.float32 and values.is_contiguous()
    if out is None:
        out = torch.empty((1,), dtype=torch.float32, device=values.device)
    _check(lib().qaq_qnorm2_quantile(_ptr(values), values.numel(), float(upper_frac), _ptr(out), _stream()), "qaq_qnorm2_quantile")
    return out


def qaq_requantize_down(cache: Cache, *, bitsK=None, bitsV=None, policy=None, ring=None, nvalid=None):
    """Lower the widths of the cached tokens in place: to the given widths [BH, n_cols] where they are lower, or to
    the widths the selection rules give now (policy for the current token count, ring [B,H,W,n_cols], nvalid)."""
    ref = bitsK if bitsK is not None else nvalid
    n_cols = ref.shape[-1]
    for t in (bitsK, bitsV, ring, nvalid):
        assert t is None or (t.is_contiguous() and t.shape[-1] == n_cols)
    pol = C.byref(policy) if policy is not None else None
    _check(lib().qaq_requantize_down(cache.handle, _ptr(bitsK), _ptr(bitsV), pol, _ptr(ring), _ptr(nvalid), n_cols,
                                     _stream()), "qaq_requantize_down")


def qaq_requantize(cache: Cache, K_full, V_full, thr, *, bitsK=None, bitsV=None, policy=None, ring=None, nvalid=None):
    """Bring every cached token to its new width, lower or higher.  K_full/V_full: the unquantized fp16 values
    [B,H,>=tokens,D] on the device or in pinned (mapped) host memory; the rest as in qaq_requantize_down."""
    sb, sh, st = _strides(K_full)
    assert _strides(V_full) == (sb, sh, st)
    ref = bitsK if bitsK is not None else nvalid
    n_cols = ref.shape[-1]
    for t in (bitsK, bitsV, ring, nvalid):
        assert t is None or (t.is_contiguous() and t.shape[-1] == n_cols)
    pol = C.byref(policy) if policy is not None else None
    _check(lib().qaq_requantize(cache.handle, _ptr(K_full), _ptr(V_full), sb, sh, st, _ptr(thr), _ptr(bitsK), _ptr(bitsV), pol,
                                _ptr(ring), _ptr(nvalid), n_cols, _stream()), "qaq_requantize")


def qaq_cache_compact(cache: Cache):
    """Close the gaps that moved tiles left in the code pools."""
    _check(lib().qaq_cache_compact(cache.handle, _stream()), "qaq_cache_compact")


def qaq_cache_pool_use(cache: Cache):
    """(largest K pool fill, largest V pool fill, pool capacity), bytes per (b,h)."""
    used = (C.c_long * 2)()
    cap = C.c_long()
    _check(lib().qaq_cache_pool_use(cache.handle, used, C.byref(cap), _stream()), "qaq_cache_pool_use")
    return int(used[0]), int(used[1]), int(cap.value)


def qaq_decode_attention(cache: Cache, q, softmax_scale, out=None, scores_out=None):
    BH, D = cache.cfg.batch * cache.cfg.heads, cache.cfg.head_dim
    assert q.dtype == torch.float16 and q.is_contiguous() and q.numel() == BH * D
    if out is None:
        out = torch.empty((BH, D), dtype=torch.float32, device=q.device)
    ws = cache.workspace()
    _check(lib().qaq_decode_attention(cache.handle, _ptr(q), float(softmax_scale), _ptr(out), _ptr(scores_out), _ptr(ws),
                                      ws.numel(), _stream()), "qaq_decode_attention")
    return out


def qaq_decode_attention_multi(cache: Cache, q, softmax_scale, out=None):
    """Several queries per (b,h): q fp16 [B*H, n_q, D] on the device; returns fp32 [B*H, n_q, D]."""
    BH, D = cache.cfg.batch * cache.cfg.heads, cache.cfg.head_dim
    assert q.dtype == torch.float16 and q.is_contiguous() and q.dim() == 3 and q.shape[0] == BH and q.shape[2] == D
    n_q = q.shape[1]
    if out is None:
        out = torch.empty((BH, n_q, D), dtype=torch.float32, device=q.device)
    nb = C.c_size_t()
    _check(lib().qaq_decode_multi_workspace_bytes(cache.handle, C.byref(nb)), "qaq_decode_multi_workspace_bytes")
    if getattr(cache, "_ws_multi", None) is None or cache._ws_multi.numel() < nb.value:
        cache._ws_multi = torch.empty(nb.value, dtype=torch.uint8, device=q.device)
    ws = cache._ws_multi
    _check(lib().qaq_decode_attention_multi(cache.handle, _ptr(q), n_q, float(softmax_scale), _ptr(out), _ptr(ws), ws.numel(),
                                            _stream()), "qaq_decode_attention_multi")
    return out


def qaq_stream_begin(cache: Cache):
    """The token count moves to device memory: from here to qaq_stream_end only the qaq_stream_* calls may be used."""
    _check(lib().qaq_stream_begin(cache.handle, _stream()), "qaq_stream_begin")


def qaq_stream_end(cache: Cache):
    """Brings the token count back to the host (synchronises the current stream); returns it."""
    _check(lib().qaq_stream_end(cache.handle, _stream()), "qaq_stream_end")
    return cache.tokens


def qaq_stream_append(cache: Cache, k_new, v_new, thr, *, bitK=None, bitV=None, policy=None, score_col=None, nvalid=None):
    """One token per (b,h) behind the device-side count: k_new / v_new fp16 [B,H,1,D] (or [B,H,D])."""
    if k_new.dim() == 3:
        k_new, v_new = k_new.unsqueeze(2), v_new.unsqueeze(2)
    assert k_new.shape[2] == 1
    sb, sh, _ = _strides(k_new)
    assert _strides(v_new)[:2] == (sb, sh)
    pol = C.byref(policy) if policy is not None else None
    _check(lib().qaq_stream_append(cache.handle, _ptr(k_new), _ptr(v_new), sb, sh, _ptr(bitK), _ptr(bitV), pol,
                                   _ptr(score_col), _ptr(nvalid), _ptr(thr), _stream()), "qaq_stream_append")


def qaq_stream_decode(cache: Cache, q, softmax_scale, out, scores_out=None):
    """Decode attention over as many tokens as the device-side count says; scores_out fp32 [B*H, >= max_tokens]."""
    BH, D = cache.cfg.batch * cache.cfg.heads, cache.cfg.head_dim
    assert q.dtype == torch.float16 and q.is_contiguous() and q.numel() == BH * D
    assert out.dtype == torch.float32 and out.is_contiguous() and out.numel() == BH * D
    stride = 0
    if scores_out is not None:
        assert scores_out.dtype == torch.float32 and scores_out.is_contiguous() and scores_out.shape[0] == BH
        stride = scores_out.shape[1]
    ws = cache.workspace()
    _check(lib().qaq_stream_decode(cache.handle, _ptr(q), float(softmax_scale), _ptr(out), _ptr(scores_out), stride, _ptr(ws),
                                   ws.numel(), _stream()), "qaq_stream_decode")
    return out


def qaq_decode_attention_static(cache: Cache, q, softmax_scale, out):
    """Decode attention that allocates nothing: the split partials live in a fixed 4 MiB device array inside
    the library instead of a workspace.  For callers that cannot obtain device memory at call time; `out`
    (float32 [B*H, D]) must already exist.  Calls share the array, so do not let two of them overlap on the GPU."""
    BH, D = cache.cfg.batch * cache.cfg.heads, cache.cfg.head_dim
    assert q.dtype == torch.float16 and q.is_contiguous() and q.numel() == BH * D
    assert out.dtype == torch.float32 and out.is_contiguous() and out.numel() == BH * D
    _check(lib().qaq_decode_attention_static(cache.handle, _ptr(q), float(softmax_scale), _ptr(out), _stream()),
           "qaq_decode_attention_static")
    return out


def qaq_quantize_append_host(cache: Cache, K_new, V_new, policy, ring, nvalid, thr):
    """All tensors on the host (pinned recommended); K_new/V_new contiguous [B,H,n,D]."""
    for t in (K_new, V_new, ring, nvalid, thr):
        assert t.device.type == "cpu" and t.is_contiguous()
    _check(lib().qaq_quantize_append_host(cache.handle, _ptr(K_new), _ptr(V_new), K_new.shape[2], C.byref(policy),
                                          _ptr(ring), _ptr(nvalid), _ptr(thr), _stream()), "qaq_quantize_append_host")


def qaq_decode_attention_host(cache: Cache, q, softmax_scale, out):
    assert q.device.type == "cpu" and out.device.type == "cpu" and q.is_contiguous() and out.is_contiguous()
    _check(lib().qaq_decode_attention_host(cache.handle, _ptr(q), float(softmax_scale), _ptr(out), _stream()),
           "qaq_decode_attention_host")
    return out


def qaq_cache_stats(cache: Cache) -> Stats:
    s = Stats()
    _check(lib().qaq_cache_stats(cache.handle, C.byref(s), _stream()), "qaq_cache_stats")
    return s


def qaq_cache_export(cache: Cache, tensor: int):
    """Canonical arrays of K (0) or V (1) as torch tensors on the device."""
    cfg = cache.cfg
    BH, D, T = cfg.batch * cfg.heads, cfg.head_dim, cache.tokens
    st = qaq_cache_stats(cache)
    dev = "cuda"
    bits = torch.empty((BH, T), dtype=torch.uint8, device=dev)
    mn = torch.empty((BH, T), dtype=torch.float32, device=dev)
    step = torch.empty((BH, T), dtype=torch.float32, device=dev)
    off = torch.empty((BH, T + 1), dtype=torch.int32, device=dev)
    rowptr = torch.empty((BH, T + 1), dtype=torch.int32, device=dev)
    cs = T * D
    os_ = max(1, int(st.outliers[tensor]))   # upper bound for any single (b,h)
    codes = torch.zeros((BH, cs), dtype=torch.uint8, device=dev)
    ch = torch.zeros((BH, os_), dtype=torch.uint8, device=dev)
    val = torch.zeros((BH, os_), dtype=torch.float16, device=dev)
    _check(lib().qaq_cache_export(cache.handle, tensor, _ptr(bits), _ptr(mn), _ptr(step), _ptr(off), _ptr(codes), cs,
                                  _ptr(rowptr), _ptr(ch), _ptr(val), os_, _stream()), "qaq_cache_export")
    return dict(bits=bits, mn=mn, step=step, off=off, codes=codes, rowptr=rowptr, ch=ch, val=val, stats=st)
