"""Pins for the oracle's LRSA attention forward and backward (Section 3.1 Eq. 3; Section 3.2
Attn-Fill 1/2).  Independent checks: a library softmax + autograd over an explicit [N,N] mask
built chunk by chunk from the text, the dense-causal special case, finite differences, a
hand-enumerated mask, and invariants of the static mask."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import lrsa_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rand_bits(shape, seed):
    g = torch.Generator().manual_seed(seed)
    return orc.bf16_bits(torch.randn(shape, generator=g).to(torch.bfloat16))


def random_idx(p, seed):
    """Any valid selection: K distinct ascending positions inside each scored window."""
    g = orc.geometry(p)
    rng = np.random.default_rng(seed)
    idx = np.zeros((p.B, p.Hkv, g["Wsel"], p.K), np.int32)
    for b in range(p.B):
        for h in range(p.Hkv):
            for w in range(g["Wsel"]):
                idx[b, h, w] = p.S + w * p.L + np.sort(rng.choice(p.L, p.K, replace=False))
    return idx


def text_mask(p, idx, b, hkv):
    """[N,N] boolean mask written chunk by chunk from the Attn-Fill description: a query chunk
    sees the sinks, the kept tokens of the compressed windows, the uncompressed windows before
    it, and itself causally."""
    N, S, L = p.N, p.S, p.L
    W = (N - S) // L if N >= S else 0
    Wsel = max(W - 1, 0)
    M = np.zeros((N, N), bool)
    for t in range(min(S, N)):          # sinks among themselves
        M[t, :t + 1] = True
    starts = list(range(S, N, L))       # chunk starts (the last chunk may be a short tail)
    for c, q0 in enumerate(starts):
        q1 = min(q0 + L, N)
        M[q0:q1, :S] = True
        ncomp = min(max(c - p.n_dense_prev, 0), Wsel)
        for w in range(c):
            if w < ncomp:
                M[q0:q1, idx[b, hkv, w]] = True
            else:
                M[q0:q1, S + w * L:S + (w + 1) * L] = True
        for t in range(q0, q1):
            M[t, q0:t + 1] = True
    return M


def torch_reference(p, Q, K, V, dO, idx):
    """softmax(QK^T*scale + M) V with a library softmax; gradients from autograd."""
    q = torch.tensor(orc.bits_to_f64(Q) if Q.dtype == np.uint16 else Q, requires_grad=True)
    k = torch.tensor(orc.bits_to_f64(K) if K.dtype == np.uint16 else K, requires_grad=True)
    v = torch.tensor(orc.bits_to_f64(V) if V.dtype == np.uint16 else V, requires_grad=True)
    go = torch.tensor(orc.bits_to_f64(dO) if dO.dtype == np.uint16 else dO)
    G = p.Hq // p.Hkv
    scale = p.scale if p.scale else 1 / math.sqrt(p.d)
    M = torch.tensor(np.stack([np.stack([text_mask(p, idx, b, h // G) for h in range(p.Hq)]) for b in range(p.B)]))
    kk = k.repeat_interleave(G, dim=1)
    vv = v.repeat_interleave(G, dim=1)
    s = (q @ kk.transpose(-1, -2)) * scale
    s = s.masked_fill(~M, -math.inf)
    O = torch.softmax(s, -1) @ vv
    lse = torch.logsumexp(s, -1)
    (O * go).sum().backward()
    return O.detach().numpy(), lse.detach().numpy(), q.grad.numpy(), k.grad.numpy(), v.grad.numpy()


CASES = [
    # B Hq Hkv N  d  L  K  S ndp
    (1, 1, 1, 9, 4, 2, 1, 1, 1),
    (1, 2, 1, 33, 8, 4, 2, 3, 1),     # tail T=2
    (2, 2, 2, 32, 8, 8, 3, 0, 1),     # S=0, T=0
    (1, 7, 1, 50, 4, 8, 2, 1, 1),     # GQA 7, tail 1
    (1, 4, 2, 45, 8, 4, 1, 3, 0),     # variant: previous window already compressed
    (1, 2, 2, 64, 8, 8, 8, 0, 1),     # K = L
    (1, 1, 1, 10, 4, 8, 2, 4, 1),     # W = 0: plain causal
    (1, 2, 1, 21, 4, 8, 4, 2, 1),     # W = 2 -> one scored window, never consumed with ndp=1
    (1, 2, 1, 40, 4, 8, 4, 0, 0),
]


@pytest.mark.parametrize("case", CASES)
def test_matches_brute_force_mask_and_autograd(case):
    B, Hq, Hkv, N, d, L, K, S, ndp = case
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S, n_dense_prev=ndp)
    Q, Kt, V, dO = (rand_bits((B, h, N, d), s) for h, s in ((Hq, 1), (Hkv, 2), (Hkv, 3), (Hq, 4)))
    idx = random_idx(p, 5)
    O, LSE = orc.attn_fwd(p, Q, Kt, V, idx)
    dQ, dK, dV = orc.attn_bwd(p, Q, Kt, V, dO, idx)
    rO, rL, rdQ, rdK, rdV = torch_reference(p, Q, Kt, V, dO, idx)
    for got, want in ((O, rO), (LSE, rL), (dQ, rdQ), (dK, rdK), (dV, rdV)):
        np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)
    # the pair predicate agrees with the chunk-by-chunk mask
    for b in range(B):
        for h in range(Hkv):
            M = text_mask(p, idx, b, h)
            for t in range(N):
                assert (orc.visible_row(p, idx, b, h, t) == M[t]).all()


def test_hand_enumerated_mask():
    rows = {}
    kept = None
    for line in open(os.path.join(GOLD, "mask_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        if k == "kept":
            kept = [int(x) for x in v]
        else:
            rows[int(k)] = np.array([c == "1" for c in v[0]])
    p = orc.OracleParams(1, 1, 1, 9, 2, 2, 1, 1)
    idx = np.array(kept, np.int32).reshape(1, 1, 3, 1)
    for t in range(9):
        assert (orc.visible_row(p, idx, 0, 0, t) == rows[t]).all(), t


def test_hand_enumerated_mask_previous_window_compressed():
    """The n_dense_prev = 0 variant against masks enumerated by hand (two cases: every window
    followed by a full one, and a tail that leaves the last window uncompressed)."""
    cases, cur = [], None
    for line in open(os.path.join(GOLD, "mask_ndp0_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        if k == "case":
            cur = {"N": int(v[2]), "S": int(v[4]), "L": int(v[6]), "K": int(v[8]), "rows": {}}
            cases.append(cur)
        elif k == "kept":
            cur["kept"] = [int(x) for x in v]
        else:
            cur["rows"][int(k)] = np.array([c == "1" for c in v[0]])
    assert len(cases) == 2
    for c in cases:
        p = orc.OracleParams(1, 1, 1, c["N"], 2, c["L"], c["K"], c["S"], n_dense_prev=0)
        wsel = orc.geometry(p)["Wsel"]
        idx = np.array(c["kept"], np.int32).reshape(1, 1, wsel, c["K"])
        assert len(c["rows"]) == c["N"]
        for t in range(c["N"]):
            assert (orc.visible_row(p, idx, 0, 0, t) == c["rows"][t]).all(), (c["N"], t)


def test_full_retention_is_dense_causal():
    """K = L keeps everything: results equal textbook causal attention for any idx."""
    B, Hq, Hkv, N, d, L, S = 1, 4, 2, 70, 16, 16, 3
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, L, S)
    Q, Kt, V, dO = (rand_bits((B, h, N, d), s) for h, s in ((Hq, 11), (Hkv, 12), (Hkv, 13), (Hq, 14)))
    idx = random_idx(p, 0)
    q, k, v, go = (torch.tensor(orc.bits_to_f64(x)) for x in (Q, Kt, V, dO))
    q.requires_grad_(); k.requires_grad_(); v.requires_grad_()
    O = torch.nn.functional.scaled_dot_product_attention(
        q, k.repeat_interleave(2, 1), v.repeat_interleave(2, 1), is_causal=True)
    (O * go).sum().backward()
    oO, _ = orc.attn_fwd(p, Q, Kt, V, idx)
    dQ, dK, dV = orc.attn_bwd(p, Q, Kt, V, dO, idx)
    np.testing.assert_allclose(oO, O.detach().numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(dQ, q.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dK, k.grad.numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(dV, v.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_finite_differences():
    """Analytic dQ/dK/dV equal central differences of sum(O * R) with the selection frozen."""
    B, Hq, Hkv, N, d, L, K, S = 1, 2, 1, 27, 4, 4, 2, 2
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S)
    rng = np.random.default_rng(3)
    Q = rng.standard_normal((B, Hq, N, d)); Kt = rng.standard_normal((B, Hkv, N, d))
    V = rng.standard_normal((B, Hkv, N, d)); R = rng.standard_normal((B, Hq, N, d))
    idx = random_idx(p, 1)
    dQ, dK, dV = orc.attn_bwd(p, Q, Kt, V, R, idx)

    def loss(q, k, v):
        return float((orc.attn_fwd(p, q, k, v, idx)[0] * R).sum())

    eps = 1e-6
    for name, X, grad in (("Q", Q, dQ), ("K", Kt, dK), ("V", V, dV)):
        for _ in range(12):
            pos = tuple(rng.integers(0, s) for s in X.shape)
            Xp, Xm = X.copy(), X.copy()
            Xp[pos] += eps; Xm[pos] -= eps
            args_p = {"Q": (Xp, Kt, V), "K": (Q, Xp, V), "V": (Q, Kt, Xp)}[name]
            args_m = {"Q": (Xm, Kt, V), "K": (Q, Xm, V), "V": (Q, Kt, Xm)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * eps)
            assert abs(fd - grad[pos]) <= 1e-7 * max(1.0, abs(fd)), (name, pos, fd, grad[pos])


def test_early_chunks_are_dense_and_unkept_rows_do_not_matter():
    B, Hq, Hkv, N, d, L, K, S = 1, 2, 1, 4 * 8 + 2 + 3, 8, 8, 2, 2
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S)
    Q, Kt, V = rand_bits((B, Hq, N, d), 1), rand_bits((B, Hkv, N, d), 2), rand_bits((B, Hkv, N, d), 3)
    idx = random_idx(p, 2)
    O, LSE = orc.attn_fwd(p, Q, Kt, V, idx)
    # positions below S + 2L see exactly the causal prefix
    pd = orc.OracleParams(B, Hq, Hkv, N, d, L, L, S)
    Od, LSEd = orc.attn_fwd(pd, Q, Kt, V, random_idx(pd, 0))
    cut = S + 2 * L
    np.testing.assert_array_equal(O[:, :, :cut], Od[:, :, :cut])
    np.testing.assert_array_equal(LSE[:, :, :cut], LSEd[:, :, :cut])
    assert np.abs(O[:, :, cut:] - Od[:, :, cut:]).max() > 1e-3
    # first row: O_0 = V_0, LSE_0 = q0.k0*scale
    np.testing.assert_allclose(O[0, :, 0], np.repeat(orc.bits_to_f64(V)[0, :, 0], Hq, 0), rtol=1e-14)
    # overwrite the un-kept rows of window 0: chunks >= 2 unchanged
    K2, V2 = Kt.copy(), V.copy()
    un = [j for j in range(S, S + L) if j not in idx[0, 0, 0]]
    K2[0, 0, un] = rand_bits((len(un), d), 77)
    V2[0, 0, un] = rand_bits((len(un), d), 78)
    O2, _ = orc.attn_fwd(p, Q, K2, V2, idx)
    np.testing.assert_array_equal(O2[:, :, cut:], O[:, :, cut:])
    assert np.abs(O2[:, :, S:cut] - O[:, :, S:cut]).max() > 1e-3


def test_unkept_rows_get_no_gradient_from_later_chunks():
    B, Hq, Hkv, N, d, L, K, S = 1, 2, 1, 5 * 8 + 1, 8, 8, 3, 1
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S)
    Q, Kt, V, dO = (rand_bits((B, h, N, d), s) for h, s in ((Hq, 1), (Hkv, 2), (Hkv, 3), (Hq, 4)))
    idx = random_idx(p, 4)
    dO = dO.copy()
    dO[:, :, :S + 2 * L] = 0          # gradient only enters through chunks >= 2
    _, dK, dV = orc.attn_bwd(p, Q, Kt, V, dO, idx)
    kept0 = set(idx[0, 0, 0].tolist())
    for j in range(S, S + L):
        if j in kept0:
            assert np.abs(dK[0, 0, j]).max() > 0 and np.abs(dV[0, 0, j]).max() > 0
        else:
            assert np.abs(dK[0, 0, j]).max() == 0 and np.abs(dV[0, 0, j]).max() == 0
    assert np.abs(dV[0, 0, :S]).max() > 0       # sinks are always seen


def test_row_subsets_equal_full():
    B, Hq, Hkv, N, d, L, K, S = 2, 4, 2, 41, 8, 8, 2, 1
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S)
    Q, Kt, V, dO = (rand_bits((B, h, N, d), s) for h, s in ((Hq, 1), (Hkv, 2), (Hkv, 3), (Hq, 4)))
    idx = random_idx(p, 6)
    O, LSE = orc.attn_fwd(p, Q, Kt, V, idx)
    dQ, dK, dV = orc.attn_bwd(p, Q, Kt, V, dO, idx)
    rows = np.array([[0, 0, 0], [1, 3, 40], [0, 2, 17], [1, 1, 9]], np.int32)
    o, l = orc.fwd_rows(p, Q, Kt, V, idx, rows)
    g = orc.bwd_rows(p, Q, Kt, V, dO, idx, rows)
    keys = np.array([[0, 0, 0], [1, 1, 40], [0, 1, 12], [1, 0, 30]], np.int32)
    gk, gv = orc.bwd_keys(p, Q, Kt, V, dO, idx, keys)
    for i, (b, h, t) in enumerate(rows):
        np.testing.assert_array_equal(o[i], O[b, h, t]); assert l[i] == LSE[b, h, t]
        np.testing.assert_array_equal(g[i], dQ[b, h, t])
    for i, (b, h, j) in enumerate(keys):
        np.testing.assert_array_equal(gk[i], dK[b, h, j])
        np.testing.assert_array_equal(gv[i], dV[b, h, j])
