"""Shared helpers of the GPU parity tests: tolerances, tie accounting, oracle plumbing."""
import os

import numpy as np
import torch

from oracle import lrsa_oracle as orc
from paper_2506_11498_b200 import lrsa, workloads

# Contract for bf16 I/O with fp32 accumulation: max-abs 2e-2 and relative L2 1e-2.  A bf16 output x
# carries a rounding error of up to |x| * 2^-9 whatever the arithmetic before it, so the absolute bound
# of an element is 2e-2 + |reference| * 2^-8 (one bf16 ulp): for |reference| <= 1 this is the plain
# 2e-2 of the contract up to 0.4e-2, for larger elements it follows the output format.
MAX_ABS = 2e-2
REL_L2 = 1e-2
BF16_ULP = 2.0 ** -8
TIE_REL = 1e-6

# One record per comparison (test id, tensor, unscaled errors); written to the file named by the
# environment variable LRSA_PARITY_REPORT when the session ends (see conftest.py).
REPORT = []


def oparams(w, **kw):
    return orc.OracleParams(w.B, w.Hq, w.Hkv, w.N, w.d, w.L, w.K, w.S, **kw)


def host_bits(host):
    return {k: orc.bf16_bits(v) for k, v in host.items()}


def error_stats(got, want):
    """Unscaled error figures of one comparison."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    err = np.abs(got - want)
    denom = np.linalg.norm(want)
    small = np.abs(want) <= 1.0
    return {"max_abs": float(err.max()) if err.size else 0.0,
            "max_abs_ref_le_1": float(err[small].max()) if small.any() else 0.0,
            "rel_l2": float(np.linalg.norm(got - want) / denom) if denom > 0 else float(np.linalg.norm(got - want)),
            "max_ref": float(np.abs(want).max()) if want.size else 0.0,
            "worst_over_bound": float((err / (MAX_ABS + BF16_ULP * np.abs(want))).max()) if err.size else 0.0,
            "n": int(err.size)}


def check_close(name, got, want, max_abs=MAX_ABS, rel_l2=REL_L2, ulp=BF16_ULP, terms=None, extra=None):
    """Element-wise |got - want| <= max_abs + ulp * |want| and relative L2 <= rel_l2.  Prints and
    records the unscaled maximum error next to the verdict.  `terms` (same shape, optional): the sum of
    the absolute terms that make up each element; ulp * terms is added to the bound (forward error of a
    sum of products with one operand rounded to bf16).  Used for one ill-conditioned case only."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    assert got.shape == want.shape, (name, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    st = error_stats(got, want)
    REPORT.append({"test": os.environ.get("PYTEST_CURRENT_TEST", ""), "tensor": name, **st})
    print(f"{name}: max|err| {st['max_abs']:.3g} (where |ref|<=1: {st['max_abs_ref_le_1']:.3g}), "
          f"rel L2 {st['rel_l2']:.3g}, max|ref| {st['max_ref']:.3g}, worst err/bound {st['worst_over_bound']:.3g}")
    err = np.abs(got - want)
    bound = max_abs + ulp * np.abs(want)
    if terms is not None:
        bound = bound + ulp * np.asarray(terms, np.float64)
    if extra is not None:          # an absolute allowance per element, derived by the caller
        bound = bound + np.asarray(extra, np.float64)
    worst = int(np.argmax(err - bound))
    assert (err <= bound).all(), f"{name}: |err|={err.flat[worst]:.4g} at {worst} (ref {want.flat[worst]:.4g})"
    assert st["rel_l2"] <= rel_l2, f"{name}: relative L2 {st['rel_l2']:.3g} > {rel_l2}"
    return st["max_abs"], st["rel_l2"]


def compare_idx(got_idx, want_idx, oracle_score, S, L):
    """Bit-exact except at oracle score ties: every position present on one side only must have an
    oracle score within TIE_REL (relative) of the oracle's K-th score of that window.
    Returns the number of windows that differ (all tolerated)."""
    got_idx = np.asarray(got_idx)
    assert got_idx.shape == want_idx.shape and got_idx.dtype == np.int32
    B, H, W, K = want_idx.shape
    differing = 0
    for b in range(B):
        for h in range(H):
            for w in range(W):
                g, o = got_idx[b, h, w], want_idx[b, h, w]
                assert (np.diff(g) > 0).all(), f"window {(b, h, w)}: not strictly ascending"
                assert g[0] >= S + w * L and g[-1] < S + (w + 1) * L, f"window {(b, h, w)}: out of window"
                if np.array_equal(g, o):
                    continue
                differing += 1
                sc = oracle_score[b, h, w]
                kth = np.sort(sc)[::-1][K - 1]
                for pos in np.setxor1d(g, o):
                    s = sc[pos - S - w * L]
                    assert abs(s - kth) <= TIE_REL * abs(kth), \
                        f"window {(b, h, w)} pos {pos}: score {s!r} vs K-th {kth!r} is not a tie"
    return differing


def to_dev(host):
    return {k: v.cuda() for k, v in host.items()}


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def gradient_error_terms(w, op, bits, oidx, oO, oL, cu=()):
    """Quantities, from the oracle's values (numpy, fp64, dense [N,N] per head: small cases only), that
    bound what the arithmetic of a bf16 tensor-core backward can do to a gradient element:
      mQ, mK, mV : sums of the absolute terms of each element of dQ, dK, dV
                     dQ[t,c] = scale * sum_j dS[t,j] K[j,c]  ->  scale * sum_j |dS[t,j]| |K[j,c]|   (dK alike with Q)
                     dV[j,c] = sum_t P[t,j] dO[t,c]           ->  sum_t P[t,j] |dO[t,c]|
                   a product whose left operand is rounded to bf16 (P and dS are, to reach the tensor
                   cores) errs by up to 2^-9 of that sum, however small the cancelled result is;
      dK_from_D  : what the rounding of O to bf16 does to dK through D = rowsum(dO * O), which the dK/dV
                   kernel takes from the stored O: delta_t (four standard deviations of a sum of d
                   independent roundings of relative size 2^-9) enters dS[t,j] as P[t,j] * delta_t, hence
                   dK[j,c] as scale * sum_t P[t,j] |delta_t| |Q[t,c]|.  It matters where a query puts most
                   of its weight on one key (the first tokens of a sequence, dominant keys)."""
    G = w.Hq // w.Hkv
    scale = 1.0 / np.sqrt(w.d)
    Q, K, V, dO = (orc.bits_to_f64(bits[k]) for k in ("Q", "K", "V", "dO"))
    mQ, mK, mV, tK = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V), np.zeros_like(K)
    for b in range(w.B):
        for hq in range(w.Hq):
            h = hq // G
            if cu:
                vis = np.stack([orc.visible_row_packed(op, oidx, cu, b, h, t) for t in range(w.N)])
            else:
                vis = np.stack([orc.visible_row(op, oidx, b, h, t) for t in range(w.N)])
            S = (Q[b, hq] @ K[b, h].T) * scale
            P = np.where(vis, np.exp(S - oL[b, hq][:, None]), 0.0)
            dP = dO[b, hq] @ V[b, h].T
            D = (P * dP).sum(-1, keepdims=True)
            dS = np.abs(P * (dP - D))
            mQ[b, hq] = scale * dS @ np.abs(K[b, h])
            mK[b, h] += scale * dS.T @ np.abs(Q[b, hq])
            mV[b, h] += P.T @ np.abs(dO[b, hq])
            delta = 4.0 * 2.0 ** -9 / np.sqrt(3.0) * np.sqrt(((dO[b, hq] * oO[b, hq]) ** 2).sum(-1, keepdims=True))
            tK[b, h] += scale * P.T @ (delta * np.abs(Q[b, hq]))
    return {"mQ": mQ, "mK": mK, "mV": mV, "dK_from_D": tK}
