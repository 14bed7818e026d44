"""Pins for the oracle's LagKV scoring and top-K selection (Section 3.2, Eq. 4-8)."""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from oracle import lrsa_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(np.asarray(x, np.float32)).to(torch.bfloat16)
    assert torch.equal(t.float(), torch.from_numpy(np.asarray(x, np.float32))), "not bf16-exact"
    return orc.bf16_bits(t)


def _rand_bits(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return orc.bf16_bits((scale * torch.randn(shape, generator=g)).to(torch.bfloat16))


def _library_score(p, K, V):
    """Eq. 4-8 restated with library routines (np.min/max, np.std, scipy softmax)."""
    g = orc.geometry(p)
    out = np.zeros((p.B, p.Hkv, g["Wsel"], p.L))
    for Z in (orc.bits_to_f64(K), orc.bits_to_f64(V)):
        body = Z[:, :, p.S:p.S + g["W"] * p.L].reshape(p.B, p.Hkv, g["W"], p.L, p.d)
        cur, nxt = body[:, :, :-1], body[:, :, 1:]
        mn = nxt.min(axis=3, keepdims=True)
        mx = nxt.max(axis=3, keepdims=True)
        rng = mx - mn
        zb = np.where(rng == 0, 0.0, (cur - mn) / np.where(rng == 0, 1.0, rng))
        out += scipy.special.softmax(zb.std(axis=-1, ddof=p.ddof), axis=-1)
    return out


def test_hand_worked_example():
    rows = {}
    for line in open(os.path.join(GOLD, "score_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        rows[k] = np.array([float(x) for x in v])
    p = orc.OracleParams(B=1, Hq=1, Hkv=1, N=4, d=2, L=2, K=1, S=0)
    K = _bits(rows["K"].reshape(1, 1, 4, 2))
    V = _bits(rows["V"].reshape(1, 1, 4, 2))
    sc, sk, sv = orc.score(p, K, V, parts=True)
    np.testing.assert_allclose(sk.ravel(), rows["score_K"], atol=1e-9)
    np.testing.assert_allclose(sv.ravel(), rows["score_V"], atol=1e-9)
    np.testing.assert_allclose(sc.ravel(), rows["score"], atol=1e-9)
    # closed form, independent of the fixture's digits
    a = 1.0 / (1.0 + math.exp(-1.0 / math.sqrt(2.0)))
    np.testing.assert_allclose(sk.ravel(), [a, 1 - a], atol=1e-14)
    assert orc.select(p, sc).ravel().tolist() == [int(rows["top1"][0])]


@pytest.mark.parametrize("B,H,N,d,L,S,ddof", [
    (1, 1, 40, 8, 8, 0, 1), (2, 3, 77, 16, 12, 5, 1), (1, 2, 300, 64, 32, 4, 0), (1, 1, 200, 128, 64, 3, 1),
])
def test_matches_library_restatement(B, H, N, d, L, S, ddof):
    p = orc.OracleParams(B=B, Hq=H, Hkv=H, N=N, d=d, L=L, K=max(L // 4, 1), S=S, ddof=ddof)
    K = _rand_bits((B, H, N, d), 1)
    V = _rand_bits((B, H, N, d), 2, scale=3.0)
    np.testing.assert_allclose(orc.score(p, K, V), _library_score(p, K, V), rtol=1e-12, atol=1e-15)


def test_sum_is_two_and_positive():
    p = orc.OracleParams(B=2, Hq=2, Hkv=2, N=150, d=32, L=16, K=4, S=6)
    sc, sk, sv = orc.score(p, _rand_bits((2, 2, 150, 32), 3), _rand_bits((2, 2, 150, 32), 4), parts=True)
    assert (sc > 0).all()
    np.testing.assert_allclose(sk.sum(-1), 1.0, atol=1e-13)
    np.testing.assert_allclose(sv.sum(-1), 1.0, atol=1e-13)
    np.testing.assert_allclose(sc.sum(-1), 2.0, atol=1e-13)


def test_affine_invariance_per_channel():
    """Eq. 6 removes any per-channel a*z+b (a>0) applied to window and reference alike."""
    rng = np.random.default_rng(0)
    B, H, N, d, L, S = 1, 2, 50, 8, 8, 2
    p = orc.OracleParams(B=B, Hq=H, Hkv=H, N=N, d=d, L=L, K=2, S=S)
    Kf = rng.integers(-32, 33, (B, H, N, d)) / 4.0
    Vf = rng.integers(-32, 33, (B, H, N, d)) / 4.0
    a = np.array([0.5, 1, 2, 4, 0.5, 2, 1, 4]).reshape(1, 1, 1, d)
    b = rng.integers(-4, 5, (1, H, 1, d)).astype(float)
    s0 = orc.score(p, _bits(Kf), _bits(Vf))
    s1 = orc.score(p, _bits(a * Kf + b), _bits(a * Vf - b))
    np.testing.assert_allclose(s0, s1, rtol=1e-12)


def test_permutation_properties():
    rng = np.random.default_rng(1)
    B, H, N, d, L, S = 1, 1, 3 * 16 + 3, 16, 16, 3
    p = orc.OracleParams(B=B, Hq=H, Hkv=H, N=N, d=d, L=L, K=4, S=S)
    K = _rand_bits((B, H, N, d), 7)
    V = _rand_bits((B, H, N, d), 8)
    s0 = orc.score(p, K, V)
    # channels permuted: unchanged
    pc = rng.permutation(d)
    np.testing.assert_allclose(orc.score(p, np.ascontiguousarray(K[..., pc]), np.ascontiguousarray(V[..., pc])), s0, rtol=1e-12)
    # tokens of the reference window (window 1) permuted: window 0's score unchanged
    pr = np.arange(N)
    pr[S + L:S + 2 * L] = S + L + rng.permutation(L)
    s_ref = orc.score(p, np.ascontiguousarray(K[:, :, pr]), np.ascontiguousarray(V[:, :, pr]))
    np.testing.assert_allclose(s_ref[:, :, 0], s0[:, :, 0], rtol=1e-12)
    # tokens of the scored window 0 permuted: window 0's score permutes with them
    perm = rng.permutation(L)
    ps = np.arange(N)
    ps[S:S + L] = S + perm
    s_perm = orc.score(p, np.ascontiguousarray(K[:, :, ps]), np.ascontiguousarray(V[:, :, ps]))
    np.testing.assert_allclose(s_perm[:, :, 0], s0[:, :, 0][..., perm], rtol=1e-12)


def test_constant_channel_contributes_zero():
    """A channel with zero reference range is read as normalised value 0 for every token."""
    B, H, N, d, L, S = 1, 1, 24, 4, 8, 0
    p = orc.OracleParams(B=B, Hq=H, Hkv=H, N=N, d=d, L=L, K=2, S=S)
    K = orc.bits_to_f64(_rand_bits((B, H, N, d), 9))
    V = orc.bits_to_f64(_rand_bits((B, H, N, d), 10))
    K[..., 1] = 2.0   # constant everywhere: range 0 in every reference window
    s = orc.score(p, _bits(K), _bits(V))
    assert np.isfinite(s).all()
    np.testing.assert_allclose(s, _library_score(p, _bits(K), _bits(V)), rtol=1e-12)
    # same result as if that channel held a constant normalised value 0
    K2 = K.copy()
    K2[..., 1] = 0.0
    # make channel 1's reference range [0,1] with all scored tokens at the minimum
    K2[:, :, L, 1] = 1.0        # one reference token of window 1 raises the max; window 0 tokens stay at min -> 0
    s2 = orc.score(p, _bits(K2), _bits(V))
    np.testing.assert_allclose(s2[:, :, 0], s[:, :, 0], rtol=1e-12)


@pytest.mark.parametrize("L,K", [(8, 1), (8, 8), (16, 5), (64, 16)])
def test_select_matches_stable_argsort(L, K):
    rng = np.random.default_rng(L * 100 + K)
    B, H, S, W = 2, 3, 5, 4
    N = S + W * L + 3
    p = orc.OracleParams(B=B, Hq=H, Hkv=H, N=N, d=8, L=L, K=K, S=S)
    sc = rng.random((B, H, W - 1, L))
    sc[0, 0, 0, :] = np.round(sc[0, 0, 0, :] * 3) / 3   # many exact ties
    idx = orc.select(p, sc)
    assert idx.shape == (B, H, W - 1, K)
    for b in range(B):
        for h in range(H):
            for w in range(W - 1):
                want = np.sort(np.argsort(-sc[b, h, w], kind="stable")[:K]) + S + w * L
                assert idx[b, h, w].tolist() == want.tolist()


def test_select_ties_go_to_lower_position():
    p = orc.OracleParams(B=1, Hq=1, Hkv=1, N=12, d=8, L=4, K=2, S=0)
    sc = np.array([[[[0.5, 0.7, 0.5, 0.5], [0.1, 0.1, 0.1, 0.1]]]])
    assert orc.select(p, sc)[0, 0].tolist() == [[0, 1], [4, 5]]


def test_geometry():
    g = orc.geometry(orc.OracleParams(1, 28, 4, 32768, 128, 1024, 256, 4))
    assert g == {"W": 31, "T": 1020, "C": 32, "Wsel": 30}
    g = orc.geometry(orc.OracleParams(1, 1, 1, 9, 2, 2, 1, 1))
    assert g == {"W": 4, "T": 0, "C": 4, "Wsel": 3}
    g = orc.geometry(orc.OracleParams(1, 1, 1, 10, 2, 8, 1, 4))
    assert g == {"W": 0, "T": 6, "C": 1, "Wsel": 0}
