"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times.

The fp64 CPU oracle cannot run a whole 32K-131K layer in seconds, so at these sizes
  * scoring/selection is compared in full (the oracle's cost is linear in N),
  * O, LSE and dQ are compared on sampled query rows, dK and dV on sampled key rows that the
    oracle can compute one by one (keys whose visible-query set is small enough),
  * and two identities that hold at any size cover every element of the gradients:
      sum_j dV_j = sum_{heads of the group} sum_t dO_t           (rows of P sum to one)
      sum_t q_t . dQ_t = sum_j k_j . dK_j   per (batch, KV group) (both are scale * sum dS_tj s_tj)
Tolerances are the contract's: indices bit-exact up to counted oracle ties, max-abs 2e-2 and
relative L2 1e-2 for bf16 outputs.
"""
import numpy as np
import pytest
import torch

from oracle import lrsa_oracle as orc
from paper_2506_11498_b200 import lrsa, workloads
from tests.parity_utils import check_close, compare_idx, f64, host_bits, oparams

pytestmark = pytest.mark.gpu


def _sample_rows(w, rng, n):
    """Query rows: fixed boundary rows (sinks, first/last row of chunks, last token) + random ones."""
    C = (w.N - w.S + w.L - 1) // w.L
    fixed = [0, max(w.S - 1, 0), w.S, w.S + w.L - 1, w.S + w.L, w.S + 2 * w.L - 1, w.S + 2 * w.L,
             w.S + (C - 1) * w.L - 1, w.S + (C - 1) * w.L, w.N - 1]
    ts = [t for t in fixed if 0 <= t < w.N] + list(rng.integers(0, w.N, n))
    rows = [(int(rng.integers(0, w.B)), int(rng.integers(0, w.Hq)), int(t)) for t in ts]
    return np.array(rows, np.int32)


def _sample_keys(w, idx, rng, n_cheap, n_kept):
    """Key rows the oracle can afford.  An un-kept key of window v is seen only by the queries from
    itself to the end of chunk v+1, so un-kept keys from the last quarter of a window cost about
    1.25 L query rows per head; half of them come from the first three windows (short rows), half
    from anywhere.  Plus the last token, the last key of the last full window, and kept keys of the
    last scored windows (seen compressed only by the final chunks)."""
    W = (w.N - w.S) // w.L
    Wsel = max(W - 1, 0)
    keys = []
    for i in range(n_cheap):
        b, h = int(rng.integers(0, w.B)), int(rng.integers(0, w.Hkv))
        kept = np.zeros(w.N, bool)
        if Wsel:
            kept[idx[b, h].reshape(-1)] = True
        v = int(rng.integers(0, min(3, W))) if i % 2 == 0 else int(rng.integers(0, W))
        lo = w.S + v * w.L + (3 * w.L) // 4
        cand = np.flatnonzero(~kept[lo:w.S + (v + 1) * w.L]) + lo
        keys.append((b, h, int(rng.choice(cand))))
    keys.append((0, 0, w.N - 1))
    keys.append((w.B - 1, w.Hkv - 1, w.S + W * w.L - 1))
    for i in range(n_kept):
        if Wsel == 0:
            break
        b, h = int(rng.integers(0, w.B)), int(rng.integers(0, w.Hkv))
        win = max(Wsel - 1 - (i % 2), 0)
        keys.append((b, h, int(idx[b, h, win, -1 - int(rng.integers(0, max(w.K // 8, 1)))])))
    return np.array(keys, np.int32)


def _identities(w, dev, dQ, dK, dV):
    G = w.Hq // w.Hkv
    # sum_j dV_j = sum over the group's heads and all t of dO_t   (fp32 sums of bf16 values)
    lhs = dV.float().sum(dim=2)
    rhs = dev["dO"].float().view(w.B, w.Hkv, G, w.N, w.d).sum(dim=(2, 3))
    scale = dev["dO"].float().abs().view(w.B, w.Hkv, G * w.N, w.d).sum(dim=2)
    # every dV element carries bf16 rounding (2^-9 relative), summed over N rows
    assert ((lhs - rhs).abs() <= 4e-3 * scale + 1e-2).all(), float(((lhs - rhs).abs() / scale).max())
    qdq = (dev["Q"].float() * dQ.float()).sum(dim=(2, 3)).view(w.B, w.Hkv, G).sum(dim=2).double()
    kdk = (dev["K"].float() * dK.float()).sum(dim=(2, 3)).double()
    mag = (dev["K"].float() * dK.float()).abs().sum(dim=(2, 3)).double()
    assert ((qdq - kdk).abs() <= 4e-3 * mag).all(), (qdq, kdk, mag)


def _run_full(w, n_rows, n_cheap_keys, n_kept_keys, ndp=1, heavy_keys=()):
    """`heavy_keys`: (batch, kv head, selector) with selector "sink0" (position 0) or "kept0" (the first
    kept position of window 0): the keys that every later chunk and all query heads of the group
    accumulate into, i.e. the longest accumulation chains of dK and dV."""
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w, n_dense_prev=ndp)
    oidx, osc = orc.score_select(op, bits["K"], bits["V"])
    dev = {k: v.cuda() for k, v in host.items()}
    p = lrsa.Params.from_workload(w, n_dense_prev=ndp)
    sizes = lrsa.lrsa_workspace_bytes(p)
    ws = [lrsa.new_workspace(s) for s in sizes]
    idx, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws[0])
    ties = compare_idx(idx.cpu().numpy(), oidx, osc, w.S, w.L)
    # the attention oracle consumes the GPU's indices, so a tolerated tie does not leak downstream
    gidx = np.ascontiguousarray(idx.cpu().numpy())
    O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx, workspace=ws[1])
    dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx, workspace=ws[2])
    torch.cuda.synchronize()
    for s in ws:
        assert lrsa.lrsa_workspace_status(s) == 0
    for t in (O, LSE, dQ, dK, dV):
        assert torch.isfinite(t).all()
    rng = np.random.default_rng(1234 + w.seed)
    rows = _sample_rows(w, rng, n_rows)
    oO, oL = orc.fwd_rows(op, bits["Q"], bits["K"], bits["V"], gidx, rows)
    odQ = orc.bwd_rows(op, bits["Q"], bits["K"], bits["V"], bits["dO"], gidx, rows)
    sel = (torch.from_numpy(rows[:, 0]).long(), torch.from_numpy(rows[:, 1]).long(), torch.from_numpy(rows[:, 2]).long())
    check_close("O rows", f64(O[sel]), oO)
    check_close("LSE rows", f64(LSE[sel]), oL, max_abs=2e-3, rel_l2=1e-4, ulp=0.0)
    check_close("dQ rows", f64(dQ[sel]), odQ)
    keys = _sample_keys(w, gidx, rng, n_cheap_keys, n_kept_keys)
    heavy = [(b, h, 0 if which == "sink0" else int(gidx[b, h, 0, 0])) for b, h, which in heavy_keys]
    if heavy:
        keys = np.concatenate([keys, np.array(heavy, np.int32)])
    odK, odV = orc.bwd_keys(op, bits["Q"], bits["K"], bits["V"], bits["dO"], gidx, keys)
    ksel = (torch.from_numpy(keys[:, 0]).long(), torch.from_numpy(keys[:, 1]).long(), torch.from_numpy(keys[:, 2]).long())
    check_close("dK keys", f64(dK[ksel]), odK)
    check_close("dV keys", f64(dV[ksel]), odV)
    _identities(w, dev, dQ, dK, dV)
    print(f"{w.name}: {ties} windows differ only at oracle ties; {len(rows)} rows, {len(keys)} keys checked")
    del dev, O, LSE, dQ, dK, dV, ws
    torch.cuda.empty_cache()


def test_cfg1_4k_full_sampled():
    # small enough for a sink key and an early kept key as well
    w = workloads.CFG1
    _run_full(w, 48, 6, 2)


def test_cfg1_4k_sink_and_early_kept_keys():
    w = workloads.CFG1
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w)
    oidx, _ = orc.score_select(op, bits["K"], bits["V"])
    dev = {k: v.cuda() for k, v in host.items()}
    p = lrsa.Params.from_workload(w)
    idx = torch.from_numpy(oidx).cuda()
    O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx)
    dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx)
    keys = np.array([(0, 0, 0), (0, 3, w.S - 1), (0, 5, int(oidx[0, 5, 0, 0])), (0, 7, int(oidx[0, 7, 1, -1]))], np.int32)
    odK, odV = orc.bwd_keys(op, bits["Q"], bits["K"], bits["V"], bits["dO"], oidx, keys)
    ksel = tuple(torch.from_numpy(keys[:, i]).long() for i in range(3))
    check_close("dK keys", f64(dK[ksel]), odK)
    check_close("dV keys", f64(dV[ksel]), odV)


def test_cfg2_32k_full_sampled():
    _run_full(workloads.CFG2, 40, 4, 2, heavy_keys=[(0, 0, "sink0"), (0, 0, "kept0")])


def test_cfg3_64k_full_sampled():
    _run_full(workloads.CFG3, 24, 2, 1, heavy_keys=[(0, 1, "sink0")])


def test_cfg4_128k_full_sampled():
    _run_full(workloads.CFG4, 12, 1, 1)


def test_cfg5_sweep_index_agreement_all_points():
    """All 20 (lag window, retention) points on one tensor set: selection against the oracle."""
    pts = workloads.sweep_points()
    host = workloads.generate(pts[0], ("K", "V"))
    bits = host_bits(host)
    K, V = host["K"].cuda(), host["V"].cuda()
    total_ties = 0
    for w in pts:
        oidx, osc = orc.score_select(oparams(w), bits["K"], bits["V"])
        idx, _ = lrsa.lrsa_score_select(lrsa.Params.from_workload(w), K, V)
        total_ties += compare_idx(idx.cpu().numpy(), oidx, osc, w.S, w.L)
    print(f"cfg5 sweep: {total_ties} windows differ only at oracle ties over {len(pts)} points")


@pytest.mark.parametrize("point", [0, 3, 16, 19])
def test_cfg5_sweep_attention_corners(point):
    _run_full(workloads.sweep_points()[point], 16, 2, 1)


@pytest.mark.parametrize("wname,ndp", [("CFG1", 1), ("CFG2", 1), ("CFG2", 0), ("CFG3", 1), ("CFG4", 1)])
def test_every_element_against_the_cuda_core_kernels(wname, ndp):
    """The oracle reaches only sampled rows at these sizes.  Every element of O, LSE, dQ, dK and dV is therefore
    also compared with the library's second implementation of the same calls: CUDA-core kernels, one warp per
    row, fp32 throughout, no tiles, no tensor memory, no pipelines (and themselves checked against the oracle on
    small shapes in test_gpu_parity).  A tile that went wrong anywhere - a ragged edge, a diagonal, a hand-off -
    shows as an error of order one.  Two implementations that each hold the contract differ by at most twice its
    bound, which is the bound used here; the comparison runs on the GPU (torch elementwise ops on the outputs).
    Config 4 (a hundredth of the keys eight times larger, seen by up to 130 000 queries each) is held to that
    bound for O and LSE only: its gradient elements are cancelling sums of very many large terms, for which
    neither implementation holds an absolute bound (the CUDA-core kernels take D = rowsum(dO * O) from the bf16 O,
    the tensor-core kernels round P and dS to bf16: 2^-9 of the sum of the absolute terms either way, see
    test_attention_fwd_bwd's ill-conditioned case); there the relative L2 difference is asserted and the
    element-wise figures are printed."""
    w = getattr(workloads, wname)
    host = workloads.generate(w)
    dev = {k: v.cuda() for k, v in host.items()}
    p = lrsa.Params.from_workload(w, n_dense_prev=ndp)
    idx, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"])
    outs = []
    for impl in (0, 1):
        lrsa.lrsa_debug_set_impl(impl)
        try:
            wsb = lrsa.lrsa_workspace_bytes(p)
            ws1, ws2 = lrsa.new_workspace(wsb[1]), lrsa.new_workspace(wsb[2])
            O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx, workspace=ws1)
            dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx, workspace=ws2)
            torch.cuda.synchronize()
            assert lrsa.lrsa_workspace_status(ws1) == 0 and lrsa.lrsa_workspace_status(ws2) == 0
            outs.append(dict(O=O, LSE=LSE, dQ=dQ, dK=dK, dV=dV))
        finally:
            lrsa.lrsa_debug_set_impl(0)
    for name in ("O", "LSE", "dQ", "dK", "dV"):
        a, b = outs[0][name].float(), outs[1][name].float()
        assert torch.isfinite(a).all(), name
        err = (a - b).abs()
        bound = 2.0 * (2e-3 if name == "LSE" else 2e-2 + 2.0 ** -8 * b.abs())
        worst = (err / bound).max().item()
        rel = (err.double().pow(2).sum() / b.double().pow(2).sum()).sqrt().item()
        over = (err > bound).sum().item()
        print(f"{wname} ndp={ndp} {name}: {err.numel()} elements, max |difference| {err.max().item():.3g}, "
              f"worst difference/bound {worst:.3g}, {over} above the bound, relative L2 {rel:.3g}")
        if wname == "CFG4" and name in ("dQ", "dK", "dV"):
            assert rel <= 1e-2, (name, rel)
        else:
            assert worst <= 1.0, (name, worst)
