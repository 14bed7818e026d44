"""GPU parity of the inference side: a condensed KV cache grown in uneven steps and decode attention over
it, against the fp64 CPU oracle.  Decoding the token at position t of a cache that holds t + 1 tokens must
give row t of the oracle's forward on the first t + 1 tokens, and the kept positions recorded in the cache
must be the oracle's selection (bit-exact up to counted ties)."""
import numpy as np
import pytest
import torch

from oracle import lrsa_oracle as orc
from paper_2506_11498_b200 import lrsa, workloads
from tests.parity_utils import check_close, compare_idx, f64, host_bits

pytestmark = pytest.mark.gpu

W = workloads.Workload

CASES = [
    (W("i_d128", 2, 4, 2, 4 + 5 * 128 + 77, 128, 128, 32, 4, seed=81), (1, 1, 2, 37, 128, 300, 5, 1)),
    (W("i_d64", 1, 4, 4, 16 + 6 * 64, 64, 64, 16, 16, seed=82), (7, 64, 1, 129)),
    (W("i_gqa7", 1, 7, 1, 3 + 4 * 200 + 50, 128, 200, 50, 3, seed=83, values="channel_offset"), (250, 1, 1, 199, 403)),
    (W("i_nosink", 1, 2, 2, 6 * 96, 64, 96, 24, 0, seed=84), (96, 96, 1, 95, 200)),
    (W("i_prefill_once", 1, 4, 2, 4 + 7 * 128 + 3, 128, 128, 64, 4, seed=85), (4 + 7 * 128 + 3,)),
    # more query heads per KV head than one pass of the decode kernel takes (16): two passes over the keys
    (W("i_gqa20", 1, 20, 1, 4 + 3 * 128 + 50, 128, 128, 32, 4, seed=88), (200, 1, 150, 87)),
    (W("i_gqa40_d64", 2, 40, 1, 2 + 3 * 64 + 9, 64, 64, 16, 2, seed=89), (100, 1, 1, 101)),
    # lag windows beyond 4096 tokens are scored by the one-slice-per-CTA kernel, here on the ring
    (W("i_long_window", 1, 2, 1, 2 + 3 * 4608 + 100, 64, 4608, 100, 2, seed=86), (5000, 4608, 1, 4000)),
]


def _oracle_row(w, bits, gidx_valid, n):
    """Row n-1 of the oracle's forward on the first n tokens, for every (batch, query head)."""
    op = orc.OracleParams(w.B, w.Hq, w.Hkv, n, w.d, w.L, w.K, w.S)
    sub = {k: np.ascontiguousarray(v[:, :, :n]) for k, v in bits.items()}
    oidx, _ = orc.score_select(op, sub["K"], sub["V"])
    nv = min(gidx_valid.shape[2], oidx.shape[2])
    oidx[:, :, :nv] = gidx_valid[:, :, :nv]     # the cache's own selection where it has one (ties are checked apart)
    rows = np.array([[b, h, n - 1] for b in range(w.B) for h in range(w.Hq)], np.int32)
    O, LSE = orc.fwd_rows(op, sub["Q"], sub["K"], sub["V"], oidx, rows)
    return O.reshape(w.B, w.Hq, w.d), LSE.reshape(w.B, w.Hq)


@pytest.mark.parametrize("w,steps", CASES, ids=lambda x: x.name if hasattr(x, "name") else None)
def test_cache_growth_and_decode(w, steps):
    host = workloads.generate(w, ("Q", "K", "V"))
    bits = host_bits(host)
    dev = {k: v.cuda() for k, v in host.items()}
    p = lrsa.Params.from_workload(w)
    cache = lrsa.KVCache(p)
    i = 0
    checked = 0
    while cache.n_tokens < w.N:
        n_new = min(steps[i % len(steps)], w.N - cache.n_tokens)
        i += 1
        lo = cache.n_tokens
        cache.append(dev["K"][:, :, lo:lo + n_new].contiguous(), dev["V"][:, :, lo:lo + n_new].contiguous())
        n = cache.n_tokens
        o, lse = cache.decode(dev["Q"][:, :, n - 1].contiguous())
        assert cache.status() == 0
        wc = cache.windows_compressed()
        gidx = cache.kept()[:, :, :wc].cpu().numpy()
        oO, oL = _oracle_row(w, bits, gidx, n)
        check_close(f"o at {n} tokens", f64(o), oO)
        check_close(f"lse at {n} tokens", f64(lse), oL, max_abs=2e-3, rel_l2=1e-4, ulp=0.0)
        checked += 1
    # the selection recorded in the cache against the oracle's on the whole sequence
    op = orc.OracleParams(w.B, w.Hq, w.Hkv, w.N, w.d, w.L, w.K, w.S)
    oidx, osc = orc.score_select(op, bits["K"], bits["V"])
    wc = cache.windows_compressed()
    assert wc == max((w.N - 1 - w.S) // w.L - 1, 0) and wc <= oidx.shape[2]
    if wc:
        ties = compare_idx(np.ascontiguousarray(cache.kept()[:, :, :wc].cpu().numpy()), oidx[:, :, :wc], osc[:, :, :wc], w.S, w.L)
        print(f"{w.name}: {checked} decode steps checked, {ties} windows differ only at oracle ties")


def test_decode_equals_forward_row():
    """The decode kernel and the training forward agree on the last row (same mask, different kernels)."""
    w = W("i_vs_fwd", 1, 8, 2, 4 + 6 * 256 + 100, 128, 256, 64, 4, seed=87)
    host = workloads.generate(w, ("Q", "K", "V"))
    dev = {k: v.cuda() for k, v in host.items()}
    p = lrsa.Params.from_workload(w)
    idx, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"])
    O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx)
    cache = lrsa.KVCache(p)
    cache.append(dev["K"], dev["V"])
    o, lse = cache.decode(dev["Q"][:, :, -1].contiguous())
    wc = cache.windows_compressed()
    assert torch.equal(cache.kept()[:, :, :wc], idx[:, :, :wc])
    assert (o.float() - O[:, :, -1].float()).abs().max().item() <= 1e-2
    assert (lse - LSE[:, :, -1]).abs().max().item() <= 1e-3


def test_cache_rejects_bad_arguments():
    p = lrsa.Params(1, 4, 2, 1000, 128, 128, 32, 4)
    cache = lrsa.KVCache(p)
    k = torch.zeros((1, 2, 8, 128), dtype=torch.bfloat16, device="cuda")
    cache.n_tokens = 996
    with pytest.raises(lrsa.LrsaError) as e:       # beyond the capacity
        cache.append(k, k)
    assert e.value.status == 1
    with pytest.raises(lrsa.LrsaError) as e:
        lrsa.KVCache(lrsa.Params(1, 4, 2, 1000, 128, 128, 32, 4, n_dense_prev=0))
    assert e.value.status == 2
