"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Indices bit-exact up to counted oracle ties; O, dQ, dK, dV within max-abs 2e-2
and relative L2 1e-2."""
import numpy as np
import pytest
import torch

from oracle import lrsa_oracle as orc
from paper_2506_11498_b200 import lrsa, workloads
from tests.parity_utils import (REPORT, check_close, gradient_error_terms, compare_idx, error_stats, f64, host_bits, oparams, to_dev)

pytestmark = pytest.mark.gpu

W = workloads.Workload

SCORE_CASES = [
    W("s_d128", 2, 4, 2, 2048 + 4 + 77, 128, 256, 64, 4, seed=11),
    W("s_d64", 1, 4, 4, 4096, 64, 512, 128, 16, seed=12),
    W("s_ragged128", 1, 2, 2, 3 + 7 * 100 + 5, 128, 100, 30, 3, seed=13),
    W("s_ragged64", 2, 2, 2, 9 * 72, 64, 72, 9, 0, seed=14),
    W("s_keepall", 1, 2, 2, 5 * 128 + 2, 128, 128, 128, 2, seed=15),
    W("s_keep1", 1, 2, 2, 5 * 128 + 2, 64, 128, 1, 2, seed=16),
    W("s_offsets", 1, 4, 2, 4 + 8 * 1024, 128, 1024, 256, 4, seed=17, values="channel_offset"),
    W("s_salient", 1, 2, 2, 4 + 4 * 2048 + 9, 128, 2048, 512, 4, seed=18, values="salient"),
    W("s_tiny_window", 1, 1, 1, 70, 64, 8, 3, 1, seed=19),
    # lag windows beyond 4096 tokens take the one-slice-per-CTA kernel with global statistics
    W("s_long_window", 1, 1, 1, 2 + 3 * 4608 + 11, 64, 4608, 100, 2, seed=42),
    W("s_long_window128", 1, 2, 1, 4 * 4160, 128, 4160, 4000, 0, seed=43),
]


@pytest.mark.parametrize("w", SCORE_CASES, ids=lambda w: w.name)
@pytest.mark.parametrize("ddof", [1, 0])
def test_score_select(w, ddof):
    if ddof == 0 and w.name not in ("s_d128", "s_d64"):
        pytest.skip("ddof=0 covered on two cases")
    host = workloads.generate(w, ("K", "V"))
    bits = host_bits(host)
    op = oparams(w, ddof=ddof)
    oidx, osc = orc.score_select(op, bits["K"], bits["V"])
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w, std_ddof=ddof)
    ws = lrsa.new_workspace(lrsa.lrsa_workspace_bytes(p)[0])
    idx, sc = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws, want_score=True)
    assert lrsa.lrsa_workspace_status(ws) == 0
    np.testing.assert_allclose(f64(sc), osc, rtol=2e-5, atol=0)
    ties = compare_idx(idx.cpu().numpy(), oidx, osc, w.S, w.L)
    print(f"{w.name}: windows differing only at oracle ties: {ties}")
    # a second call on the same workspace gives the same bits
    idx2, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws)
    assert torch.equal(idx, idx2)


def test_score_zero_range_channel():
    w = W("s_const", 1, 2, 2, 2 + 4 * 128, 128, 128, 32, 2, seed=20)
    host = workloads.generate(w, ("K", "V"))
    host["K"][..., 5] = 1.5
    host["V"][:, 0, :, 100] = -2.0
    bits = host_bits(host)
    oidx, osc = orc.score_select(oparams(w), bits["K"], bits["V"])
    dev = to_dev(host)
    idx, sc = lrsa.lrsa_score_select(lrsa.Params.from_workload(w), dev["K"], dev["V"], want_score=True)
    np.testing.assert_allclose(f64(sc), osc, rtol=2e-5)
    compare_idx(idx.cpu().numpy(), oidx, osc, w.S, w.L)


ATTN_CASES = [
    # name, B, Hq, Hkv, N, d, L, K, S ; then ndp
    (W("a_d128", 1, 4, 2, 4 + 5 * 256 + 77, 128, 256, 64, 4, seed=21), 1),
    (W("a_d64", 2, 4, 4, 16 + 6 * 128, 64, 128, 32, 16, seed=22), 1),           # T = 0
    (W("a_gqa7", 1, 7, 1, 3 + 4 * 200 + 50, 128, 200, 50, 3, seed=23), 1),      # L, S not tile multiples
    (W("a_nosink", 1, 2, 2, 5 * 128 + 1, 64, 128, 100, 0, seed=24), 1),         # S = 0, T = 1
    (W("a_keepall", 1, 2, 1, 4 + 4 * 128 + 30, 128, 128, 128, 4, seed=25), 1),  # K = L: dense causal
    (W("a_ndp0", 1, 4, 2, 4 + 5 * 256 + 77, 128, 256, 64, 4, seed=26), 0),
    (W("a_short", 1, 2, 2, 300, 128, 256, 64, 4, seed=27), 1),                  # W = 1: plain causal
    (W("a_two", 1, 2, 2, 4 + 2 * 256 + 10, 64, 256, 16, 4, seed=28), 1),        # one scored window, unused
    (W("a_ndp0_two", 1, 2, 2, 4 + 2 * 256 + 10, 64, 256, 16, 4, seed=29), 0),
    (W("a_one_token", 1, 1, 1, 1, 64, 8, 2, 0, seed=30), 1),
    (W("a_sinks_only", 1, 2, 1, 5, 64, 8, 2, 5, seed=31), 1),
    (W("a_offsets", 1, 4, 2, 4 + 5 * 256 + 77, 128, 256, 64, 4, seed=32, values="channel_offset"), 1),
    (W("a_salient64", 1, 4, 1, 16 + 5 * 128 + 40, 64, 128, 32, 16, seed=33, values="salient"), 1),
]


def _run_attention(w, ndp, idx_np, host, impl=0):
    """impl 0: the tensor-core kernels; 1: the CUDA-core validation kernels (fp32 throughout)."""
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w, n_dense_prev=ndp)
    idx = torch.from_numpy(idx_np).cuda()
    wf, wb = lrsa.lrsa_workspace_bytes(p)[1:]
    wsf, wsb = lrsa.new_workspace(wf), lrsa.new_workspace(wb)
    lrsa.lrsa_debug_set_impl(impl)
    try:
        O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx, workspace=wsf)
        dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx, workspace=wsb)
    finally:
        lrsa.lrsa_debug_set_impl(0)
    assert lrsa.lrsa_workspace_status(wsf) == 0 and lrsa.lrsa_workspace_status(wsb) == 0
    return O, LSE, dQ, dK, dV


@pytest.mark.parametrize("w,ndp", ATTN_CASES, ids=lambda x: x.name if hasattr(x, "name") else str(x))
def test_attention_fwd_bwd(w, ndp):
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w, n_dense_prev=ndp)
    oidx, _ = orc.score_select(op, bits["K"], bits["V"])
    oO, oL = orc.attn_fwd(op, bits["Q"], bits["K"], bits["V"], oidx)
    odQ, odK, odV = orc.attn_bwd(op, bits["Q"], bits["K"], bits["V"], bits["dO"], oidx)
    O, LSE, dQ, dK, dV = _run_attention(w, ndp, oidx, host)
    check_close("O", f64(O), oO)
    check_close("LSE", f64(LSE), oL, max_abs=2e-3, rel_l2=1e-4, ulp=0.0)
    if w.values == "salient":
        # The deliberately ill-conditioned case (700 tokens, d = 64, a handful of keys scaled by 8): its
        # gradient elements are cancelling sums of large terms, and the bound follows the terms.
        e = gradient_error_terms(w, op, bits, oidx, oO, oL)
        check_close("dQ", f64(dQ), odQ, terms=e["mQ"])
        check_close("dK", f64(dK), odK, terms=e["mK"], extra=e["dK_from_D"])
        check_close("dV", f64(dV), odV, terms=e["mV"])
    else:
        check_close("dQ", f64(dQ), odQ)
        check_close("dK", f64(dK), odK)
        check_close("dV", f64(dV), odV)


@pytest.mark.parametrize("name", ["a_salient64", "a_offsets", "a_gqa7", "a_ndp0"])
def test_cuda_core_validation_kernels_against_oracle(name):
    """The slow CUDA-core kernels (fp32 P and dS, no tensor cores) against the oracle at the same
    element-wise bound: they share the bf16 inputs and outputs with the tensor-core path but none of its
    bf16 rounding of P and dS, so their error is the floor set by the I/O format alone."""
    w, ndp = next(c for c in ATTN_CASES if c[0].name == name)
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w, n_dense_prev=ndp)
    oidx, _ = orc.score_select(op, bits["K"], bits["V"])
    oO, oL = orc.attn_fwd(op, bits["Q"], bits["K"], bits["V"], oidx)
    odQ, odK, odV = orc.attn_bwd(op, bits["Q"], bits["K"], bits["V"], bits["dO"], oidx)
    O, LSE, dQ, dK, dV = _run_attention(w, ndp, oidx, host, impl=1)
    check_close("ref-kernel O", f64(O), oO)
    check_close("ref-kernel LSE", f64(LSE), oL, max_abs=2e-3, rel_l2=1e-4, ulp=0.0)
    check_close("ref-kernel dV", f64(dV), odV)
    if name == "a_salient64":
        # These kernels take D = rowsum(dO * O) from the bf16 O, as the textbook backward does.  With a few
        # dominant keys of large norm that D is not accurate enough for dQ and dK, fp32 arithmetic or not:
        # the error is recorded (it is why the tensor-core path sums P * dP instead), not bounded.
        for nm, got, want in (("dQ", dQ, odQ), ("dK", dK, odK)):
            st = error_stats(f64(got), want)
            REPORT.append({"test": "textbook D, fp32 CUDA-core kernels, a_salient64", "tensor": nm, **st})
            print(f"ref-kernel {nm} with the textbook D: max|err| {st['max_abs']:.3g}, rel L2 {st['rel_l2']:.3g}")
            assert st["rel_l2"] < 2e-2
        assert error_stats(f64(dQ), odQ)["max_abs"] > 2e-2
    else:
        check_close("ref-kernel dQ", f64(dQ), odQ)
        check_close("ref-kernel dK", f64(dK), odK)


def test_end_to_end_and_determinism():
    w = W("e2e", 2, 8, 2, 4 + 6 * 256 + 100, 128, 256, 64, 4, seed=40, values="channel_offset")
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w)
    oidx, osc = orc.score_select(op, bits["K"], bits["V"])
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w)
    idx, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"])
    assert compare_idx(idx.cpu().numpy(), oidx, osc, w.S, w.L) == 0
    outs = []
    for _ in range(2):
        O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx)
        dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx)
        outs.append((O, LSE, dQ, dK, dV))
    rows = orc.all_rows(op)[:: 37]
    oO, oL = orc.fwd_rows(op, bits["Q"], bits["K"], bits["V"], oidx, rows)
    got = np.stack([f64(outs[0][0][b, h, t]) for b, h, t in rows])
    check_close("O rows", got, oO)
    # run-to-run: forward bitwise, backward within accumulation-order noise
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    for a, b in zip(outs[0][2:], outs[1][2:]):
        assert (a.float() - b.float()).abs().max().item() <= 2e-2


def test_unkept_rows_get_no_gradient_from_later_chunks():
    """Static-mask invariant: with dO zero before chunk 2, un-kept rows of window 0 get exactly zero
    dK and dV while its kept rows and the sinks do not."""
    w = W("p11", 1, 4, 2, 4 + 5 * 256, 128, 256, 64, 4, seed=41)
    host = workloads.generate(w)
    host["dO"][:, :, : w.S + 2 * w.L] = 0
    bits = host_bits(host)
    oidx, _ = orc.score_select(oparams(w), bits["K"], bits["V"])
    O, LSE, dQ, dK, dV = _run_attention(w, 1, oidx, host)
    kept = np.zeros(w.N, bool)
    kept[oidx[0, 0, 0]] = True
    win0 = np.arange(w.S, w.S + w.L)
    un = win0[~kept[win0]]
    assert dK[0, 0, un].abs().max().item() == 0 and dV[0, 0, un].abs().max().item() == 0
    assert dV[0, 0, oidx[0, 0, 0]].abs().min(dim=0).values.max().item() > 0
    assert dV[0, 0, : w.S].abs().max().item() > 0


# ---- packed variable-length batches and query chunks of several lag windows ----

PACKED_CASES = [
    # workload (N = last boundary), boundaries, ndp
    (W("p_two", 1, 4, 2, 1500, 128, 128, 32, 4, seed=51), (0, 4 + 5 * 128 + 77, 1500), 1),     # unequal, both with tails
    (W("p_three64", 2, 4, 4, 1200, 64, 64, 16, 16, seed=52), (0, 16 + 8 * 64, 16 + 8 * 64 + 10, 1200), 1),  # T = 0; shorter than S
    (W("p_gqa7", 1, 7, 1, 1000, 128, 100, 30, 3, seed=53, values="channel_offset"), (0, 333, 334, 1000), 1),  # one-token sequence
    (W("p_ndp0", 1, 2, 2, 900, 64, 128, 32, 4, seed=54), (0, 500, 900), 0),
]


@pytest.mark.parametrize("w,cu,ndp", PACKED_CASES, ids=lambda x: x.name if hasattr(x, "name") else None)
def test_packed_sequences(w, cu, ndp):
    """Several sequences back to back on the token axis: every stage against the oracle applied to
    each sequence on its own."""
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w, n_dense_prev=ndp)
    oidx, osc = orc.score_select_packed(op, bits["K"], bits["V"], cu)
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w, n_dense_prev=ndp, cu_seqlens=cu)
    assert lrsa.lrsa_num_sel_windows(p) == oidx.shape[2]
    sizes = lrsa.lrsa_workspace_bytes(p)
    ws = [lrsa.new_workspace(s) for s in sizes]
    idx, sc = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws[0], want_score=True)
    np.testing.assert_allclose(f64(sc), osc, rtol=2e-5, atol=0)
    got = idx.cpu().numpy()
    for t0, n, wsel, woff in orc.packed_windows(op, cu):      # per sequence: window numbering restarts
        if wsel:
            compare_idx(got[:, :, woff:woff + wsel] - t0, oidx[:, :, woff:woff + wsel] - t0,
                        osc[:, :, woff:woff + wsel], min(w.S, n), w.L)
    idx = torch.from_numpy(oidx).cuda()
    O, LSE = lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx, workspace=ws[1])
    dQ, dK, dV = lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx, workspace=ws[2])
    for s in ws:
        assert lrsa.lrsa_workspace_status(s) == 0
    oO, oL = orc.attn_fwd_packed(op, bits["Q"], bits["K"], bits["V"], oidx, cu)
    odQ, odK, odV = orc.attn_bwd_packed(op, bits["Q"], bits["K"], bits["V"], bits["dO"], oidx, cu)
    check_close("O", f64(O), oO)
    check_close("LSE", f64(LSE), oL, max_abs=2e-3, rel_l2=1e-4, ulp=0.0)
    check_close("dQ", f64(dQ), odQ)
    check_close("dK", f64(dK), odK)
    check_close("dV", f64(dV), odV)


def test_packed_single_sequence_equals_unpacked():
    w = W("p_one", 1, 4, 2, 4 + 5 * 256 + 77, 128, 256, 64, 4, seed=55)
    dev = to_dev(workloads.generate(w))
    a = lrsa.Params.from_workload(w)
    b = lrsa.Params.from_workload(w, cu_seqlens=(0, w.N))
    ia, _ = lrsa.lrsa_score_select(a, dev["K"], dev["V"])
    ib, _ = lrsa.lrsa_score_select(b, dev["K"], dev["V"])
    assert torch.equal(ia, ib)
    Oa, La = lrsa.lrsa_attn_fwd(a, dev["Q"], dev["K"], dev["V"], ia)
    Ob, Lb = lrsa.lrsa_attn_fwd(b, dev["Q"], dev["K"], dev["V"], ia)
    assert torch.equal(Oa, Ob) and torch.equal(La, Lb)


@pytest.mark.parametrize("m", [2, 4])
def test_query_chunk_of_several_lag_windows(m):
    """chunk = m * lag: the mask does not depend on how many windows are filled at a time, so the
    results are those of chunk = lag (and match the oracle, which has no chunk parameter)."""
    w = W("c_multi", 1, 4, 2, 4 + 6 * 128 + 50, 128, 128, 32, 4, seed=56)
    host = workloads.generate(w)
    bits = host_bits(host)
    op = oparams(w)
    oidx, _ = orc.score_select(op, bits["K"], bits["V"])
    oO, _ = orc.attn_fwd(op, bits["Q"], bits["K"], bits["V"], oidx)
    dev = to_dev(host)
    p1 = lrsa.Params.from_workload(w)
    pm = lrsa.Params.from_workload(w, chunk=m * w.L)
    i1, _ = lrsa.lrsa_score_select(p1, dev["K"], dev["V"])
    im, _ = lrsa.lrsa_score_select(pm, dev["K"], dev["V"])
    assert torch.equal(i1, im) and np.array_equal(im.cpu().numpy(), oidx)
    O1, L1 = lrsa.lrsa_attn_fwd(p1, dev["Q"], dev["K"], dev["V"], i1)
    Om, Lm = lrsa.lrsa_attn_fwd(pm, dev["Q"], dev["K"], dev["V"], im)
    assert torch.equal(O1, Om) and torch.equal(L1, Lm)
    check_close("O", f64(Om), oO)
    g1 = lrsa.lrsa_attn_bwd(p1, dev["Q"], dev["K"], dev["V"], O1, dev["dO"], L1, i1)
    gm = lrsa.lrsa_attn_bwd(pm, dev["Q"], dev["K"], dev["V"], Om, dev["dO"], Lm, im)
    odQ, odK, odV = orc.attn_bwd(op, bits["Q"], bits["K"], bits["V"], bits["dO"], oidx)
    for name, a, b, ref in zip(("dQ", "dK", "dV"), g1, gm, (odQ, odK, odV)):
        check_close(name, f64(b), ref)
        assert (a.float() - b.float()).abs().max().item() <= 2e-2


def test_expired_wait_is_reported_and_the_next_call_is_clean():
    """The bounded wait of the long-window scoring kernel, made to give up at once through the test hook:
    the call returns, the workspace reports LRSA_ERR_TIMEOUT, and an ordinary call on the same workspace
    afterwards is clean and correct."""
    w = W("s_timeout", 1, 1, 1, 2 + 3 * 4608 + 11, 64, 4608, 100, 2, seed=42)
    host = workloads.generate(w, ("K", "V"))
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w)
    ws = lrsa.new_workspace(lrsa.lrsa_workspace_bytes(p)[0])
    want, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws)
    assert lrsa.lrsa_workspace_status(ws) == 0
    lrsa.lrsa_debug_set_wait_limit(-1)
    try:
        lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws)
        assert lrsa.lrsa_workspace_status(ws) == 5      # LRSA_ERR_TIMEOUT
    finally:
        lrsa.lrsa_debug_set_wait_limit(0)
    again, _ = lrsa.lrsa_score_select(p, dev["K"], dev["V"], workspace=ws)
    assert lrsa.lrsa_workspace_status(ws) == 0
    assert torch.equal(again, want)


def _padded(shape, dtype, fill, pad=4096):
    """A tensor of `shape` carved out of a larger buffer whose margins hold a sentinel."""
    n = int(np.prod(shape))
    buf = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
    return buf, buf[pad:pad + n].view(shape)


def _margins_intact(buf, n, fill, pad=4096):
    ref = torch.full((pad,), fill, dtype=buf.dtype, device="cuda")
    return torch.equal(buf[:pad], ref) and torch.equal(buf[pad + n:], ref)


@pytest.mark.parametrize("w", [
    W("canary_ragged", 1, 7, 1, 3 + 4 * 200 + 50, 128, 200, 50, 3, seed=61),      # nothing is a tile multiple
    W("canary_d64", 2, 4, 2, 16 + 6 * 128 + 1, 64, 128, 32, 16, seed=62),
], ids=lambda w: w.name)
def test_outputs_never_written_outside_their_tensors(w):
    """Every output tensor sits inside a larger buffer with sentinel margins: after the three calls the
    margins are untouched (a stray store of a ragged tile, a bulk copy of a partial row or a reduction onto a
    wrong row would show) and every element inside has been overwritten."""
    host = workloads.generate(w)
    dev = to_dev(host)
    p = lrsa.Params.from_workload(w)
    wsel = lrsa.lrsa_num_sel_windows(p)
    bf, f32 = torch.bfloat16, torch.float32
    bi, idx = _padded((w.B, w.Hkv, wsel, w.K), torch.int32, -7)
    bs, sc = _padded((w.B, w.Hkv, wsel, w.L), f32, -7.0)
    bO, O = _padded((w.B, w.Hq, w.N, w.d), bf, 777.0)
    bL, LSE = _padded((w.B, w.Hq, w.N), f32, 777.0)
    bQ, dQ = _padded((w.B, w.Hq, w.N, w.d), bf, 777.0)
    bK, dK = _padded((w.B, w.Hkv, w.N, w.d), bf, 777.0)
    bV, dV = _padded((w.B, w.Hkv, w.N, w.d), bf, 777.0)
    lrsa.lrsa_score_select(p, dev["K"], dev["V"], idx=idx, score=sc)
    lrsa.lrsa_attn_fwd(p, dev["Q"], dev["K"], dev["V"], idx, O=O, LSE=LSE)
    lrsa.lrsa_attn_bwd(p, dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, idx, dQ=dQ, dK=dK, dV=dV)
    torch.cuda.synchronize()
    for name, buf, t, fill in (("idx", bi, idx, -7), ("score", bs, sc, -7.0), ("O", bO, O, 777.0), ("LSE", bL, LSE, 777.0),
                               ("dQ", bQ, dQ, 777.0), ("dK", bK, dK, 777.0), ("dV", bV, dV, 777.0)):
        assert _margins_intact(buf, t.numel(), fill), f"{name}: a margin was written"
        assert not (t == fill).any(), f"{name}: an element was left unwritten"
