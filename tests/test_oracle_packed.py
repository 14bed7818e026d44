"""Pins for the oracle's packed variable-length functions (several sequences back to back on the token
axis, each an independent LRSA problem): a hand-enumerated two-sequence mask, a library softmax +
autograd over an explicit block-diagonal [N,N] mask, and a library restatement of the scores per slice."""
import os

import numpy as np
import pytest
import torch

from oracle import lrsa_oracle as orc
from tests.test_oracle_attention import rand_bits, text_mask
from tests.test_oracle_score import _library_score, _rand_bits

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_hand_enumerated_packed_mask():
    rows, kept, cu = {}, None, None
    for line in open(os.path.join(GOLD, "mask_packed_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        if k == "cu":
            cu = [int(x) for x in v]
        elif k == "kept":
            kept = [int(x) for x in v]
        else:
            rows[int(k)] = np.array([c == "1" for c in v[0]])
    p = orc.OracleParams(1, 1, 1, cu[-1], 2, 2, 1, 1)
    assert [s[2] for s in orc.packed_windows(p, cu)] == [1, 3]
    idx = np.array(kept, np.int32).reshape(1, 1, 4, 1)
    for t in range(cu[-1]):
        assert (orc.visible_row_packed(p, idx, cu, 0, 0, t) == rows[t]).all(), t


def _random_packed_idx(p, cu, seed):
    rng = np.random.default_rng(seed)
    seqs = orc.packed_windows(p, cu)
    idx = np.zeros((p.B, p.Hkv, sum(s[2] for s in seqs), p.K), np.int32)
    for t0, n, wsel, woff in seqs:
        for b in range(p.B):
            for h in range(p.Hkv):
                for w in range(wsel):
                    idx[b, h, woff + w] = t0 + p.S + w * p.L + np.sort(rng.choice(p.L, p.K, replace=False))
    return idx


@pytest.mark.parametrize("cu,S,L,K,ndp", [
    ([0, 21, 30, 64], 2, 4, 2, 1),       # tails, a short sequence with one scored window
    ([0, 3, 40], 4, 8, 3, 1),            # first sequence shorter than the sink count
    ([0, 33, 66], 1, 8, 2, 0),           # variant with the previous window compressed
    ([0, 17], 1, 4, 1, 1),               # one sequence: equals the unpacked functions
])
def test_packed_matches_block_diagonal_brute_force(cu, S, L, K, ndp):
    B, Hq, Hkv, d = 1, 4, 2, 8
    N = cu[-1]
    p = orc.OracleParams(B, Hq, Hkv, N, d, L, K, S, n_dense_prev=ndp)
    Q, Kt, V, dO = (rand_bits((B, h, N, d), s) for h, s in ((Hq, 1), (Hkv, 2), (Hkv, 3), (Hq, 4)))
    idx = _random_packed_idx(p, cu, 9)
    O, LSE = orc.attn_fwd_packed(p, Q, Kt, V, idx, cu)
    dQ, dK, dV = orc.attn_bwd_packed(p, Q, Kt, V, dO, idx, cu)
    # explicit mask: each sequence's chunk-by-chunk mask on the diagonal, nothing off it
    G = Hq // Hkv
    M = np.zeros((B, Hq, N, N), bool)
    for t0, n, wsel, woff in orc.packed_windows(p, cu):
        ps = orc.OracleParams(B, Hq, Hkv, n, d, L, K, S, n_dense_prev=ndp)
        loc = np.ascontiguousarray(idx[:, :, woff:woff + wsel] - t0)
        for b in range(B):
            for h in range(Hq):
                M[b, h, t0:t0 + n, t0:t0 + n] = text_mask(ps, loc, b, h // G)
    q, k, v = (torch.tensor(orc.bits_to_f64(x), requires_grad=True) for x in (Q, Kt, V))
    s = (q @ k.repeat_interleave(G, 1).transpose(-1, -2)) / np.sqrt(d)
    s = s.masked_fill(~torch.tensor(M), -np.inf)
    o = torch.softmax(s, -1) @ v.repeat_interleave(G, 1)
    (o * torch.tensor(orc.bits_to_f64(dO))).sum().backward()
    for got, want in ((O, o.detach().numpy()), (LSE, torch.logsumexp(s, -1).detach().numpy()),
                      (dQ, q.grad.numpy()), (dK, k.grad.numpy()), (dV, v.grad.numpy())):
        np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)
    for t in range(N):
        assert (orc.visible_row_packed(p, idx, cu, 0, 1, t) == M[0, 2, t]).all()
    # row / key subsets agree with the full functions
    rows = np.array([[0, 1, 0], [0, 3, N - 1], [0, 2, min(cu[1], N - 1)], [0, 0, max(cu[1] - 1, 0)]], np.int32)
    o_r, l_r = orc.fwd_rows_packed(p, Q, Kt, V, idx, cu, rows)
    g_r = orc.bwd_rows_packed(p, Q, Kt, V, dO, idx, cu, rows)
    keys = np.array([[0, 0, 0], [0, 1, N - 1], [0, 1, min(cu[1], N - 1)]], np.int32)
    gk, gv = orc.bwd_keys_packed(p, Q, Kt, V, dO, idx, cu, keys)
    for i, (b, h, t) in enumerate(rows):
        np.testing.assert_array_equal(o_r[i], O[b, h, t]); assert l_r[i] == LSE[b, h, t]
        np.testing.assert_array_equal(g_r[i], dQ[b, h, t])
    for i, (b, h, j) in enumerate(keys):
        np.testing.assert_array_equal(gk[i], dK[b, h, j]); np.testing.assert_array_equal(gv[i], dV[b, h, j])


def test_packed_scores_use_only_their_own_sequence():
    B, H, d, L, S, Kk = 2, 2, 16, 8, 3, 2
    cu = [0, 45, 52, 120]
    p = orc.OracleParams(B, H, H, cu[-1], d, L, Kk, S)
    K, V = _rand_bits((B, H, cu[-1], d), 5), _rand_bits((B, H, cu[-1], d), 6, scale=2.0)
    idx, sc = orc.score_select_packed(p, K, V, cu)
    seqs = orc.packed_windows(p, cu)
    assert [s[2] for s in seqs] == [4, 0, 7]
    for t0, n, wsel, woff in seqs:
        if wsel == 0:
            continue
        ps = orc.OracleParams(B, H, H, n, d, L, Kk, S)
        want = _library_score(ps, np.ascontiguousarray(K[:, :, t0:t0 + n]), np.ascontiguousarray(V[:, :, t0:t0 + n]))
        np.testing.assert_allclose(sc[:, :, woff:woff + wsel], want, rtol=1e-12, atol=1e-15)
        # kept positions: stable top-K of each window, as packed positions inside that window
        for w in range(wsel):
            order = np.argsort(-want[0, 1, w], kind="stable")[:Kk]
            assert idx[0, 1, woff + w].tolist() == sorted((t0 + S + w * L + order).tolist())
    # changing another sequence's tokens changes nothing here
    K2 = K.copy(); K2[:, :, 45:52] = _rand_bits((B, H, 7, d), 7)
    idx2, sc2 = orc.score_select_packed(p, K2, V, cu)
    np.testing.assert_array_equal(sc2, sc); np.testing.assert_array_equal(idx2, idx)
