"""Thin binding over the C ABI of ``liblrsa.so`` (declared in ``include/lrsa.h``).

Argument marshalling only: torch supplies device memory and streams, every step of the path
runs in the library's CUDA kernels.  There is no fallback: if the shared library is missing
the import of any entry point raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblrsa.so")

STATUS = {0: "LRSA_OK", 1: "LRSA_ERR_INVALID_ARG", 2: "LRSA_ERR_UNSUPPORTED",
          3: "LRSA_ERR_WORKSPACE_TOO_SMALL", 4: "LRSA_ERR_CUDA", 5: "LRSA_ERR_TIMEOUT"}


class LrsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS.get(status, status)} ({status_string(status)})")


class lrsa_params_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("batch", "n_q_heads", "n_kv_heads", "seq_len", "head_dim", "chunk", "lag", "top_k",
                 "n_sink", "n_dense_prev", "std_ddof")] + [("softmax_scale", ctypes.c_float),
                                                           ("n_seqs", ctypes.c_int32),
                                                           ("cu_seqlens", ctypes.POINTER(ctypes.c_int32)),
                                                           ("o_residual", ctypes.c_void_p)]


@dataclass(frozen=True)
class Params:
    """Mirror of ``lrsa_params_t`` (Section 3.2: sink size S, lag L, kept tokens K = r*L)."""
    batch: int
    n_q_heads: int
    n_kv_heads: int
    seq_len: int
    head_dim: int
    lag: int
    top_k: int
    n_sink: int
    chunk: int = 0            # 0 -> lag
    n_dense_prev: int = 1
    std_ddof: int = 1
    softmax_scale: float = 0.0
    cu_seqlens: tuple = ()    # packed batch: boundaries (0, ..., seq_len) of the sequences on the token axis

    def c(self, o_residual=None) -> lrsa_params_t:
        """The C struct; `o_residual`: a bf16 tensor shaped like O (or None), see lrsa_attn_fwd."""
        cp = lrsa_params_t(self.batch, self.n_q_heads, self.n_kv_heads, self.seq_len, self.head_dim,
                           self.chunk or self.lag, self.lag, self.top_k, self.n_sink,
                           self.n_dense_prev, self.std_ddof, self.softmax_scale, 0, None,
                           None if o_residual is None else o_residual.data_ptr())
        if self.cu_seqlens:
            arr = (ctypes.c_int32 * len(self.cu_seqlens))(*self.cu_seqlens)
            cp.n_seqs = len(self.cu_seqlens) - 1
            cp.cu_seqlens = ctypes.cast(arr, ctypes.POINTER(ctypes.c_int32))
            cp._keepalive = arr          # the host array lives as long as the struct
        return cp

    @staticmethod
    def from_workload(w, **kw) -> "Params":
        return Params(w.B, w.Hq, w.Hkv, w.N, w.d, w.L, w.K, w.S, **kw)


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32p, fp = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(lrsa_params_t)
        L.lrsa_num_sel_windows.argtypes = [pp, ctypes.POINTER(ctypes.c_int32)]
        L.lrsa_workspace_bytes.argtypes = [pp] + [ctypes.POINTER(sz)] * 3
        L.lrsa_score_select.argtypes = [pp, vp, vp, i32p, fp, vp, sz, vp]
        L.lrsa_score_select_static.argtypes = [pp, vp, vp, i32p, fp, vp]
        L.lrsa_score_select_static.restype = ctypes.c_int
        L.lrsa_attn_fwd.argtypes = [pp, vp, vp, vp, i32p, vp, fp, vp, sz, vp]
        L.lrsa_attn_bwd.argtypes = [pp, vp, vp, vp, vp, vp, fp, i32p, vp, vp, vp, vp, sz, vp]
        i32 = ctypes.c_int32
        L.lrsa_cache_bytes.argtypes = [pp, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.lrsa_cache_append.argtypes = [pp, vp, sz, vp, vp, i32, i32, vp, sz, vp]
        L.lrsa_cache_kept.argtypes = [pp, vp, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(i32)]
        L.lrsa_attn_decode.argtypes = [pp, vp, sz, vp, i32, vp, fp, vp, sz, vp]
        for name in ("lrsa_cache_bytes", "lrsa_cache_append", "lrsa_cache_kept", "lrsa_attn_decode"):
            getattr(L, name).restype = ctypes.c_int
        L.lrsa_workspace_status.argtypes = [vp, vp]
        L.lrsa_score_select_static_status.argtypes = [vp]
        L.lrsa_score_select_static_status.restype = ctypes.c_int
        L.lrsa_status_string.argtypes = [ctypes.c_int]
        L.lrsa_status_string.restype = ctypes.c_char_p
        L.lrsa_last_launch_count.argtypes = []
        L.lrsa_debug_set_impl.argtypes = [ctypes.c_int]
        L.lrsa_debug_set_wait_limit.argtypes = [ctypes.c_int]
        L.lrsa_debug_set_wait_limit.restype = ctypes.c_int
        for name in ("lrsa_num_sel_windows", "lrsa_workspace_bytes", "lrsa_score_select", "lrsa_attn_fwd",
                     "lrsa_attn_bwd", "lrsa_workspace_status", "lrsa_last_launch_count", "lrsa_debug_set_impl"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().lrsa_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise LrsaError(status, where)


def _p(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def lrsa_num_sel_windows(params: Params) -> int:
    out = ctypes.c_int32(0)
    cp = params.c()
    _check(lib().lrsa_num_sel_windows(ctypes.byref(cp), ctypes.byref(out)), "lrsa_num_sel_windows")
    return out.value


def lrsa_workspace_bytes(params: Params):
    a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    cp = params.c()
    _check(lib().lrsa_workspace_bytes(ctypes.byref(cp), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "lrsa_workspace_bytes")
    return a.value, b.value, c.value


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def lrsa_score_select(params: Params, K, V, idx=None, score=None, workspace=None, stream=None,
                      want_score: bool = False):
    """Eq. 4-8 + top-K.  Returns (idx int32 [B,Hkv,W_sel,K], score or None)."""
    wsel = lrsa_num_sel_windows(params)
    if idx is None:
        idx = torch.empty((params.batch, params.n_kv_heads, wsel, params.top_k), dtype=torch.int32, device=K.device)
    if score is None and want_score:
        score = torch.empty((params.batch, params.n_kv_heads, wsel, params.lag), dtype=torch.float32, device=K.device)
    if workspace is None:
        workspace = new_workspace(lrsa_workspace_bytes(params)[0], K.device)
    cp = params.c()
    _check(lib().lrsa_score_select(ctypes.byref(cp), _p(K), _p(V), _p(idx), _p(score), _p(workspace),
                                   workspace.numel(), _stream(stream)), "lrsa_score_select")
    return idx, score


STATIC_SCRATCH_BYTES = 4 << 20


def lrsa_score_select_static(params: Params, K, V, idx, score=None, stream=None):
    """lrsa_score_select for callers that cannot provide or allocate scratch memory: the library's
    own fixed device array (STATIC_SCRATCH_BYTES) is used, so nothing is allocated here either -
    `idx` (and `score`, if wanted) must be passed in.  Problems that need more scratch raise
    LRSA_ERR_WORKSPACE_TOO_SMALL.  Calls that may overlap on the GPU must be serialised."""
    cp = params.c()
    _check(lib().lrsa_score_select_static(ctypes.byref(cp), _p(K), _p(V), _p(idx), _p(score), _stream(stream)),
           "lrsa_score_select_static")
    return idx, score


def lrsa_score_select_static_status(stream=None) -> int:
    """Status of the last lrsa_score_select_static call on the current device (0 = ok, 5 = a bounded
    device-side wait expired).  Synchronises the stream."""
    return lib().lrsa_score_select_static_status(_stream(stream))


def lrsa_attn_fwd(params: Params, Q, K, V, idx, O=None, LSE=None, workspace=None, stream=None, o_residual=None):
    """Eq. 3 under the chunked mask.  Returns (O bf16 [B,Hq,N,d], LSE fp32 [B,Hq,N]).  `o_residual` (bf16,
    shaped like O, optional) receives what the bf16 O cannot hold; lrsa_attn_bwd takes it to form dK more accurately."""
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None:
        LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device=Q.device)
    if workspace is None:
        workspace = new_workspace(lrsa_workspace_bytes(params)[1], Q.device)
    cp = params.c(o_residual)
    _check(lib().lrsa_attn_fwd(ctypes.byref(cp), _p(Q), _p(K), _p(V), _p(idx), _p(O), _p(LSE), _p(workspace),
                               workspace.numel(), _stream(stream)), "lrsa_attn_fwd")
    return O, LSE


def lrsa_attn_bwd(params: Params, Q, K, V, O, dO, LSE, idx, dQ=None, dK=None, dV=None, workspace=None,
                  stream=None, o_residual=None):
    """Gradient of Eq. 3 with the mask constant.  Returns (dQ, dK, dV) in bf16."""
    if dQ is None:
        dQ = torch.empty_like(Q)
    if dK is None:
        dK = torch.empty_like(K)
    if dV is None:
        dV = torch.empty_like(V)
    if workspace is None:
        workspace = new_workspace(lrsa_workspace_bytes(params)[2], Q.device)
    cp = params.c(o_residual)
    _check(lib().lrsa_attn_bwd(ctypes.byref(cp), _p(Q), _p(K), _p(V), _p(O), _p(dO), _p(LSE), _p(idx), _p(dQ),
                               _p(dK), _p(dV), _p(workspace), workspace.numel(), _stream(stream)), "lrsa_attn_bwd")
    return dQ, dK, dV


def lrsa_workspace_status(workspace, stream=None) -> int:
    return lib().lrsa_workspace_status(_p(workspace), _stream(stream))


def lrsa_last_launch_count() -> int:
    return lib().lrsa_last_launch_count()


def lrsa_debug_set_wait_limit(polls: int):
    """Test hook: polls granted to the long-window scoring kernel's wait (negative: give up at once, 0: default)."""
    _check(lib().lrsa_debug_set_wait_limit(int(polls)), "lrsa_debug_set_wait_limit")


def lrsa_debug_set_impl(impl: int):
    _check(lib().lrsa_debug_set_impl(int(impl)), "lrsa_debug_set_impl")


class KVCache:
    """Condensed KV cache of one layer for inference (Section 3.2): owns the device buffer and the token
    count; every operation runs in the library's kernels."""

    def __init__(self, params: Params, device="cuda"):
        self.params = params
        a, b = ctypes.c_size_t(0), ctypes.c_size_t(0)
        cp = params.c()
        _check(lib().lrsa_cache_bytes(ctypes.byref(cp), ctypes.byref(a), ctypes.byref(b)), "lrsa_cache_bytes")
        self.buf = torch.zeros(a.value, dtype=torch.uint8, device=device)
        self.ws = new_workspace(b.value, device)
        self.n_tokens = 0

    def append(self, k_new, v_new, stream=None):
        """k_new, v_new: bf16 [B, Hkv, n_new, d] (contiguous)."""
        n_new = k_new.shape[2]
        cp = self.params.c()
        _check(lib().lrsa_cache_append(ctypes.byref(cp), _p(self.buf), self.buf.numel(), _p(k_new), _p(v_new),
                                       self.n_tokens, n_new, _p(self.ws), self.ws.numel(), _stream(stream)),
               "lrsa_cache_append")
        self.n_tokens += n_new

    def decode(self, q, o=None, lse=None, stream=None):
        """q: bf16 [B, Hq, d], the query of the last token in the cache.  Returns (o, lse)."""
        if o is None:
            o = torch.empty_like(q)
        if lse is None:
            lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
        cp = self.params.c()
        _check(lib().lrsa_attn_decode(ctypes.byref(cp), _p(self.buf), self.buf.numel(), _p(q), self.n_tokens, _p(o),
                                      _p(lse), _p(self.ws), self.ws.numel(), _stream(stream)), "lrsa_attn_decode")
        return o, lse

    def kept(self):
        """int32 [B, Hkv, w_cap, top_k] view of the kept positions (windows compressed so far are valid)."""
        ptr, wcap = ctypes.c_void_p(0), ctypes.c_int32(0)
        cp = self.params.c()
        _check(lib().lrsa_cache_kept(ctypes.byref(cp), _p(self.buf), ctypes.byref(ptr), ctypes.byref(wcap)),
               "lrsa_cache_kept")
        off = ptr.value - self.buf.data_ptr()
        n = self.params.batch * self.params.n_kv_heads * wcap.value * self.params.top_k
        return self.buf[off:off + 4 * n].view(torch.int32).view(self.params.batch, self.params.n_kv_heads, wcap.value,
                                                                 self.params.top_k)

    def windows_compressed(self) -> int:
        p = self.params
        if self.n_tokens <= p.n_sink:
            return 0
        return max((self.n_tokens - 1 - p.n_sink) // p.lag - 1, 0)

    def status(self, stream=None) -> int:
        return lrsa_workspace_status(self.ws, stream)
