"""ctypes front end of the fp64 CPU oracle (``lrsa_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's cpu-baseline
leg load this; the CUDA library never does, and this module imports nothing from it.
Only argument marshalling lives here; all arithmetic is in the C++ file, which follows
Section 3.1 (Eq. 3) and Section 3.2 (Eq. 4-8, Attn-Fill 1/2) of the paper.

Tensors are numpy arrays.  Q/K/V/dO are bf16 bit patterns as ``uint16`` arrays of shape
``[B, H, N, d]`` (``bf16_bits`` converts a ``torch.bfloat16`` tensor without rounding), or
``float64`` arrays of the same shape (all of one kind per call).
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lrsa_oracle.cpp")
_LIB = os.path.join(_HERE, "liblrsa_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O3, OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O3", "-std=c++17", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC]
        )
    return _LIB


class _CParams(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "Hq", "Hkv", "N", "d", "L", "K", "S", "n_dense_prev", "ddof")] + \
               [("scale", ctypes.c_double)]


@dataclass(frozen=True)
class OracleParams:
    B: int
    Hq: int
    Hkv: int
    N: int
    d: int
    L: int          # lag window = query chunk
    K: int          # kept tokens per window (r * L)
    S: int          # sink tokens
    n_dense_prev: int = 1
    ddof: int = 1
    scale: float = 0.0   # 0 -> 1/sqrt(d)

    def c(self) -> _CParams:
        sc = self.scale if self.scale != 0.0 else 1.0 / math.sqrt(self.d)
        return _CParams(self.B, self.Hq, self.Hkv, self.N, self.d, self.L, self.K, self.S,
                        self.n_dense_prev, self.ddof, sc)


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.lrsa_oracle_num_threads.restype = ctypes.c_int
    return _lib


def _fn(name: str, *arrays):
    """Pick the bf16-bit or the double entry point from the arrays' dtype."""
    kinds = {a.dtype for a in arrays}
    assert len(kinds) == 1, kinds
    kind = kinds.pop()
    assert kind in (np.uint16, np.float64), kind
    return getattr(_load(), name + ("_f64" if kind == np.float64 else ""))


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def bf16_bits(t) -> np.ndarray:
    """torch.bfloat16 CPU tensor -> uint16 numpy array holding the same bits."""
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(a: np.ndarray) -> np.ndarray:
    """Exact bf16 bits -> float64 (for tests that need the values)."""
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def num_threads() -> int:
    return int(_load().lrsa_oracle_num_threads())


def geometry(p: OracleParams) -> dict:
    out = np.zeros(4, np.int32)
    cp = p.c()
    _load().lrsa_oracle_geometry(ctypes.byref(cp), _ptr(out))
    return {"W": int(out[0]), "T": int(out[1]), "C": int(out[2]), "Wsel": int(out[3])}


def score(p: OracleParams, K: np.ndarray, V: np.ndarray, parts: bool = False):
    """Eq. 4-8.  Returns score [B,Hkv,Wsel,L] (and the K and V terms if ``parts``)."""
    g = geometry(p)
    shape = (p.B, p.Hkv, g["Wsel"], p.L)
    sc = np.zeros(shape, np.float64)
    sk = np.zeros(shape, np.float64) if parts else None
    sv = np.zeros(shape, np.float64) if parts else None
    cp = p.c()
    _fn("lrsa_oracle_score", K, V)(ctypes.byref(cp), _ptr(K), _ptr(V), _ptr(sc),
                              _ptr(sk) if parts else None, _ptr(sv) if parts else None)
    return (sc, sk, sv) if parts else sc


def select(p: OracleParams, sc: np.ndarray) -> np.ndarray:
    """Top-K positions of every scored window: int32 [B,Hkv,Wsel,K], ascending."""
    g = geometry(p)
    idx = np.zeros((p.B, p.Hkv, g["Wsel"], p.K), np.int32)
    cp = p.c()
    _load().lrsa_oracle_select(ctypes.byref(cp), _ptr(np.ascontiguousarray(sc)), _ptr(idx))
    return idx


def score_select(p: OracleParams, K: np.ndarray, V: np.ndarray):
    sc = score(p, K, V)
    return select(p, sc), sc


def visible_row(p: OracleParams, idx: np.ndarray, b: int, hkv: int, t: int) -> np.ndarray:
    out = np.zeros(p.N, np.uint8)
    cp = p.c()
    _load().lrsa_oracle_visible_row(ctypes.byref(cp), _ptr(idx), b, hkv, t, _ptr(out))
    return out.astype(bool)


def all_rows(p: OracleParams) -> np.ndarray:
    b, h, t = np.meshgrid(np.arange(p.B), np.arange(p.Hq), np.arange(p.N), indexing="ij")
    return np.ascontiguousarray(np.stack([b, h, t], -1).reshape(-1, 3).astype(np.int32))


def all_keys(p: OracleParams) -> np.ndarray:
    b, h, t = np.meshgrid(np.arange(p.B), np.arange(p.Hkv), np.arange(p.N), indexing="ij")
    return np.ascontiguousarray(np.stack([b, h, t], -1).reshape(-1, 3).astype(np.int32))


def fwd_rows(p, Q, K, V, idx, rows):
    rows = np.ascontiguousarray(rows, np.int32)
    n = rows.shape[0]
    O = np.zeros((n, p.d), np.float64)
    LSE = np.zeros(n, np.float64)
    cp = p.c()
    _fn("lrsa_oracle_fwd_rows", Q, K, V)(ctypes.byref(cp), _ptr(Q), _ptr(K), _ptr(V), _ptr(idx),
                                 ctypes.c_long(n), _ptr(rows), _ptr(O), _ptr(LSE))
    return O, LSE


def bwd_rows(p, Q, K, V, dO, idx, rows):
    rows = np.ascontiguousarray(rows, np.int32)
    n = rows.shape[0]
    dQ = np.zeros((n, p.d), np.float64)
    cp = p.c()
    _fn("lrsa_oracle_bwd_rows", Q, K, V, dO)(ctypes.byref(cp), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(idx),
                                 ctypes.c_long(n), _ptr(rows), _ptr(dQ))
    return dQ


def bwd_keys(p, Q, K, V, dO, idx, keys):
    keys = np.ascontiguousarray(keys, np.int32)
    n = keys.shape[0]
    dK = np.zeros((n, p.d), np.float64)
    dV = np.zeros((n, p.d), np.float64)
    cp = p.c()
    _fn("lrsa_oracle_bwd_keys", Q, K, V, dO)(ctypes.byref(cp), _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(idx),
                                 ctypes.c_long(n), _ptr(keys), _ptr(dK), _ptr(dV))
    return dK, dV


def attn_fwd(p, Q, K, V, idx):
    """Full forward: O [B,Hq,N,d], LSE [B,Hq,N]."""
    O, LSE = fwd_rows(p, Q, K, V, idx, all_rows(p))
    return O.reshape(p.B, p.Hq, p.N, p.d), LSE.reshape(p.B, p.Hq, p.N)


def attn_bwd(p, Q, K, V, dO, idx):
    """Full backward: dQ [B,Hq,N,d], dK, dV [B,Hkv,N,d]."""
    dQ = bwd_rows(p, Q, K, V, dO, idx, all_rows(p)).reshape(p.B, p.Hq, p.N, p.d)
    dK, dV = bwd_keys(p, Q, K, V, dO, idx, all_keys(p))
    return dQ, dK.reshape(p.B, p.Hkv, p.N, p.d), dV.reshape(p.B, p.Hkv, p.N, p.d)


# ----------------------------------------------------------------------------------------------
# Packed variable-length batches.  Several sequences lie back to back along the token axis of every
# [B, H, N, d] tensor; `cu` (length n_seqs + 1, cu[0] = 0, cu[-1] = N) holds their boundaries.  Each
# sequence is an independent LRSA problem with its own sinks and lag windows counted from its own first
# token (Section 3.2 describes one sequence; nothing crosses a boundary), so every function below is
# the single-sequence function applied to each slice, with positions shifted by the slice's start.
# Scored windows are numbered sequence after sequence; kept positions are positions in the packed axis.
# ----------------------------------------------------------------------------------------------

def _seq(p: OracleParams, n: int) -> OracleParams:
    from dataclasses import replace
    return replace(p, N=int(n))


def _slice(a: np.ndarray, lo: int, hi: int) -> np.ndarray:
    return np.ascontiguousarray(a[:, :, lo:hi])


def packed_windows(p: OracleParams, cu) -> list:
    """Per sequence: (first token, length, scored windows, index of its first scored window)."""
    out, woff = [], 0
    for s in range(len(cu) - 1):
        n = int(cu[s + 1] - cu[s])
        wsel = geometry(_seq(p, n))["Wsel"]
        out.append((int(cu[s]), n, wsel, woff))
        woff += wsel
    return out


def score_select_packed(p: OracleParams, K: np.ndarray, V: np.ndarray, cu):
    seqs = packed_windows(p, cu)
    total = sum(s[2] for s in seqs)
    idx = np.zeros((p.B, p.Hkv, total, p.K), np.int32)
    sc = np.zeros((p.B, p.Hkv, total, p.L), np.float64)
    for t0, n, wsel, woff in seqs:
        if wsel == 0:
            continue
        i, s = score_select(_seq(p, n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n))
        idx[:, :, woff:woff + wsel] = i + t0
        sc[:, :, woff:woff + wsel] = s
    return idx, sc


def _local_idx(idx: np.ndarray, t0: int, wsel: int, woff: int) -> np.ndarray:
    return np.ascontiguousarray(idx[:, :, woff:woff + wsel] - t0).astype(np.int32)


def visible_row_packed(p: OracleParams, idx: np.ndarray, cu, b: int, hkv: int, t: int) -> np.ndarray:
    out = np.zeros(int(cu[-1]), bool)
    for t0, n, wsel, woff in packed_windows(p, cu):
        if t0 <= t < t0 + n:
            out[t0:t0 + n] = visible_row(_seq(p, n), _local_idx(idx, t0, wsel, woff), b, hkv, t - t0)
    return out


def attn_fwd_packed(p, Q, K, V, idx, cu):
    O = np.zeros((p.B, p.Hq, int(cu[-1]), p.d), np.float64)
    LSE = np.zeros((p.B, p.Hq, int(cu[-1])), np.float64)
    for t0, n, wsel, woff in packed_windows(p, cu):
        o, l = attn_fwd(_seq(p, n), _slice(Q, t0, t0 + n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n),
                        _local_idx(idx, t0, wsel, woff))
        O[:, :, t0:t0 + n] = o
        LSE[:, :, t0:t0 + n] = l
    return O, LSE


def attn_bwd_packed(p, Q, K, V, dO, idx, cu):
    N = int(cu[-1])
    dQ = np.zeros((p.B, p.Hq, N, p.d), np.float64)
    dK = np.zeros((p.B, p.Hkv, N, p.d), np.float64)
    dV = np.zeros((p.B, p.Hkv, N, p.d), np.float64)
    for t0, n, wsel, woff in packed_windows(p, cu):
        q, k, v = attn_bwd(_seq(p, n), _slice(Q, t0, t0 + n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n),
                           _slice(dO, t0, t0 + n), _local_idx(idx, t0, wsel, woff))
        dQ[:, :, t0:t0 + n] = q
        dK[:, :, t0:t0 + n] = k
        dV[:, :, t0:t0 + n] = v
    return dQ, dK, dV


def _by_sequence(p, cu, rows):
    """Groups (b, h, t) triples by the sequence that holds t: yields (sequence, positions in `rows`)."""
    rows = np.asarray(rows, np.int32)
    for seq in packed_windows(p, cu):
        sel = np.flatnonzero((rows[:, 2] >= seq[0]) & (rows[:, 2] < seq[0] + seq[1]))
        if sel.size:
            yield seq, sel


def fwd_rows_packed(p, Q, K, V, idx, cu, rows):
    rows = np.asarray(rows, np.int32)
    O = np.zeros((len(rows), p.d), np.float64)
    LSE = np.zeros(len(rows), np.float64)
    for (t0, n, wsel, woff), sel in _by_sequence(p, cu, rows):
        loc = rows[sel].copy()
        loc[:, 2] -= t0
        O[sel], LSE[sel] = fwd_rows(_seq(p, n), _slice(Q, t0, t0 + n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n),
                                    _local_idx(idx, t0, wsel, woff), loc)
    return O, LSE


def bwd_rows_packed(p, Q, K, V, dO, idx, cu, rows):
    rows = np.asarray(rows, np.int32)
    dQ = np.zeros((len(rows), p.d), np.float64)
    for (t0, n, wsel, woff), sel in _by_sequence(p, cu, rows):
        loc = rows[sel].copy()
        loc[:, 2] -= t0
        dQ[sel] = bwd_rows(_seq(p, n), _slice(Q, t0, t0 + n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n),
                           _slice(dO, t0, t0 + n), _local_idx(idx, t0, wsel, woff), loc)
    return dQ


def bwd_keys_packed(p, Q, K, V, dO, idx, cu, keys):
    keys = np.asarray(keys, np.int32)
    dK = np.zeros((len(keys), p.d), np.float64)
    dV = np.zeros((len(keys), p.d), np.float64)
    for (t0, n, wsel, woff), sel in _by_sequence(p, cu, keys):
        loc = keys[sel].copy()
        loc[:, 2] -= t0
        dK[sel], dV[sel] = bwd_keys(_seq(p, n), _slice(Q, t0, t0 + n), _slice(K, t0, t0 + n), _slice(V, t0, t0 + n),
                                    _slice(dO, t0, t0 + n), _local_idx(idx, t0, wsel, woff), loc)
    return dK, dV
