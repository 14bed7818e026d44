#!/usr/bin/env python
"""Benchmark of the LRSA hot path: score/select + attention forward + backward on one layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole path (lrsa_score_select, lrsa_attn_fwd, lrsa_attn_bwd) over one
batch of seeded synthetic bf16 tensors shaped like a 32K-token post-training sequence of a
7B-class GQA layer.  Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU checker
under oracle/ on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "lrsa_fwd_bwd_effective_tflops"
UNIT = "TFLOP/s"


def geometry(w, ndp=1):
    W = (w.N - w.S) // w.L
    T = w.N - w.S - W * w.L
    C = W + (1 if T > 0 else 0)
    return W, T, C, max(W - 1, 0)


def count_pairs(w, ndp=1) -> int:
    """Unmasked (query, key) pairs per query head: sinks causal among themselves; a query of chunk c
    sees S sinks, K kept keys from each compressed window, the uncompressed windows before it, and
    its own chunk causally."""
    W, T, C, Wsel = geometry(w, ndp)
    pairs = w.S * (w.S + 1) // 2
    for c in range(C):
        n_c = w.L if c < W else T
        nh = min(max(c - ndp, 0), Wsel)
        pairs += n_c * (w.S + nh * w.K + (c - nh) * w.L) + n_c * (n_c + 1) // 2
    return pairs


def flops(w, ndp=1, cu=()):
    """Effective FLOPs: 4*d per pair forward (QK^T, PV), 10*d backward (five products).  Packed batch:
    the pairs of every sequence on its own."""
    if cu:
        pairs = sum(count_pairs(w.with_(N=b - a, S=min(w.S, b - a)), ndp) for a, b in zip(cu[:-1], cu[1:]))
    else:
        pairs = count_pairs(w, ndp)
    p = pairs * w.Hq * w.B
    return 4 * w.d * p, 10 * w.d * p


def kv_bytes(w):
    Wsel = geometry(w)[3]
    return 2 * w.B * w.Hkv * w.N * w.d * 2 + w.B * w.Hkv * Wsel * w.K * 4


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        m = json.load(open(path))
        return {"hbm_gbs": m["hbm_gbs"], "bf16_tflops": m["bf16_tflops"],
                "bf16_tflops_sustained": m.get("bf16_tflops_sustained", m["bf16_tflops"]),
                "sustained_sm_mhz": (m.get("clocks_under_load") or {}).get("sm_mhz_median"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sustained_sm_mhz": 1300.0,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            busy = [x for x in sm if x > 0]
            out["sm_mhz"] = statistics.median(busy) if busy else None
            out["sm_max_mhz"] = max(mx)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


def oracle_sample(w, n_chunks=3, host=None):
    """Times the fp64 CPU checker, as it stands, on a bounded sample of workload `w`: the first
    S + n_chunks*L tokens of KV-head group 0 of batch element 0 (all of its query heads).  Attention
    is causal, so this prefix is a self-contained part of the workload: its outputs equal the
    full run's.  Returns the seconds of each leg and the effective FLOPs the sample covers."""
    import numpy as np
    from oracle import lrsa_oracle as orc
    from paper_2506_11498_b200 import workloads
    host = host if host is not None else workloads.generate(w)
    G = w.Hq // w.Hkv
    n = min(w.N, w.S + n_chunks * w.L)
    sub = w.with_(name=w.name + "_prefix", B=1, Hq=G, Hkv=1, N=n)
    bits = {k: np.ascontiguousarray(orc.bf16_bits(v)[:1, :(G if k in ("Q", "dO") else 1), :n]) for k, v in host.items()}
    op = orc.OracleParams(sub.B, sub.Hq, sub.Hkv, sub.N, sub.d, sub.L, sub.K, sub.S)
    t0 = time.perf_counter()
    idx, _ = orc.score_select(op, bits["K"], bits["V"])
    t_score = time.perf_counter() - t0
    t0 = time.perf_counter()
    orc.attn_fwd(op, bits["Q"], bits["K"], bits["V"], idx)
    t_fwd = time.perf_counter() - t0
    t0 = time.perf_counter()
    orc.attn_bwd(op, bits["Q"], bits["K"], bits["V"], bits["dO"], idx)
    t_bwd = time.perf_counter() - t0
    f_fwd, f_bwd = flops(sub)
    total = t_score + t_fwd + t_bwd
    return {"t_score": t_score, "t_fwd": t_fwd, "t_bwd": t_bwd, "seconds": total,
            "tflops": (f_fwd + f_bwd) / total / 1e12, "tokens_per_s": n / total / w.Hkv,
            "cores": orc.num_threads(),
            "sample": f"first {n} tokens (sinks + {n_chunks} chunks) of KV group 0 of batch 0 of {w.name}: "
                      f"{G} query heads, full score/select + forward + backward, {total:.1f} s of CPU work"}


def run_reference(args, w):
    """Reference arm: the CPU checker on host cores, each step a bounded sample."""
    from paper_2506_11498_b200 import replicas, workloads
    if replicas.env_rank_world()[0] != 0:
        return
    f_fwd, f_bwd = flops(w)
    vals = []
    host = workloads.generate(w)
    for i in range(args.warmup + args.steps):
        s = oracle_sample(w, n_chunks=2, host=host)
        if i >= args.warmup:
            vals.append(s)
    value = statistics.mean(v["tflops"] for v in vals)
    proj = (f_fwd + f_bwd) / (value * 1e12)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": proj * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d, "L": w.L,
                   "K": w.K, "S": w.S, "note": "each step is a bounded sample; ms_per_step is the whole-workload time at the sample's rate"},
        "tokens_per_s": w.B * w.N / proj,
        "sample_seconds_per_step": statistics.mean(v["seconds"] for v in vals),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                         "sample": vals[-1]["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# DRAM bytes per backward call (dK/dV + dQ kernels: dram__bytes_read.sum + dram__bytes_write.sum of one launch
# each) from the ncu summary under profiles/, per workload; a workload without a capture of the current
# kernels carries null
BWD_DRAM_BYTES = {"cfg2_32k_gqa7_d128": 3.080e9}


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` outside a launcher: start N ranks of this script (one per GPU, NCCL
    rendezvous on the loopback address) and pass their exit code on.  Rank 0 prints the JSON line."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def decode_leg(lrsa, torch, wl, p, dev, flush, peaks):
    """Inference side of the same layer: the condensed cache is filled with the workload's K/V, then one
    decode step (the query of the last token over sinks + kept rows + ring) is timed with L2 flushed, and
    one cache growth step of a whole lag window (which scores and condenses one window)."""
    cache = lrsa.KVCache(p)
    n0 = wl.N - wl.L - 1                      # leave room for one more window of growth
    cache.append(dev["K"][:, :, :n0].contiguous(), dev["V"][:, :, :n0].contiguous())
    q = dev["Q"][:, :, n0 - 1].contiguous()
    o = torch.empty_like(q)
    lse = torch.empty(q.shape[:2], dtype=torch.float32, device="cuda")
    ts = []
    for i in range(13):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); cache.decode(q, o, lse); e1.record(); torch.cuda.synchronize()
        if i >= 3:
            ts.append(e0.elapsed_time(e1))
    c = (n0 - 1 - wl.S) // wl.L
    keys = wl.S + max(c - 1, 0) * wl.K + (n0 - 1 - (wl.S + max(c - 1, 0) * wl.L) + 1)
    nbytes = wl.B * wl.Hkv * keys * wl.d * 2 * 2
    ms = statistics.median(ts)
    kn = dev["K"][:, :, n0:n0 + wl.L].contiguous(); vn = dev["V"][:, :, n0:n0 + wl.L].contiguous()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush.zero_(); e0.record(); cache.append(kn, vn); e1.record(); torch.cuda.synchronize()
    if cache.status() != 0:
        raise SystemExit("decode leg: the cache workspace reports a timeout")
    return {"tokens_in_cache": n0, "keys_per_kv_head": keys, "cache_rows_per_kv_head": wl.S + max(c - 1, 0) * wl.K + 2 * wl.L,
            "decode_us": ms * 1e3, "decode_gbs": nbytes / (ms * 1e-3) / 1e9,
            "decode_frac_of_hbm": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "append_one_window_us": e0.elapsed_time(e1) * 1e3}


def parity_sample(w, wl_host, dev_out, idx_dev, n_dense_prev):
    """A quick look at parity inside the benchmark record: the selection of the timed run against the
    fp64 CPU checker (windows that differ, all of which must be ties), and the unscaled maximum error of a
    few sampled rows of O and dQ.  The full comparison lives in tests/; this is a record, not a gate."""
    import numpy as np
    from oracle import lrsa_oracle as orc
    bits = {k: orc.bf16_bits(v) for k, v in wl_host.items()}
    op = orc.OracleParams(w.B, w.Hq, w.Hkv, w.N, w.d, w.L, w.K, w.S, n_dense_prev=n_dense_prev)
    oidx, osc = orc.score_select(op, bits["K"], bits["V"])
    gidx = np.ascontiguousarray(idx_dev.cpu().numpy())
    differing, not_ties = 0, 0
    for b in range(w.B):
        for h in range(w.Hkv):
            for win in range(oidx.shape[2]):
                if np.array_equal(gidx[b, h, win], oidx[b, h, win]):
                    continue
                differing += 1
                sc = osc[b, h, win]
                kth = np.sort(sc)[::-1][w.K - 1]
                for pos in np.setxor1d(gidx[b, h, win], oidx[b, h, win]):
                    if abs(sc[pos - w.S - win * w.L] - kth) > 1e-6 * abs(kth):
                        not_ties += 1
    rng = np.random.default_rng(7)
    rows = np.array([[int(rng.integers(0, w.B)), int(rng.integers(0, w.Hq)), int(t)]
                     for t in (0, w.S + w.L, w.N // 2, w.N - 1)], np.int32)
    oO, _ = orc.fwd_rows(op, bits["Q"], bits["K"], bits["V"], gidx, rows)
    odQ = orc.bwd_rows(op, bits["Q"], bits["K"], bits["V"], bits["dO"], gidx, rows)
    O, dQ = dev_out
    gO = np.stack([O[b, h, t].float().cpu().numpy() for b, h, t in rows])
    gdQ = np.stack([dQ[b, h, t].float().cpu().numpy() for b, h, t in rows])
    return {"idx_windows": int(oidx.shape[0] * oidx.shape[1] * oidx.shape[2]), "idx_windows_differing": differing,
            "idx_differences_that_are_not_ties": not_ties, "sampled_rows": len(rows),
            "max_abs_err_O": float(np.abs(gO - oO).max()), "max_abs_err_dQ": float(np.abs(gdQ - odQ).max())}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_32k_gqa7_d128",
                    help="a configuration name (cfg1_..cfg4_) or a sweep point such as cfg5_L1024_r1/4")
    ap.add_argument("--n-dense-prev", type=int, default=1, choices=[0, 1],
                    help="1: the window before the query chunk is seen uncompressed (the paper); 0: compressed too")
    ap.add_argument("--cu-seqlens", default="",
                    help="packed batch: comma-separated boundaries on the token axis, e.g. 0,16384,28672,32768")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="skip the inference-side leg (condensed cache + decode)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    from paper_2506_11498_b200 import workloads
    w = {**workloads.CONFIGS, **{pt.name: pt for pt in workloads.sweep_points()}}[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    cu = tuple(int(x) for x in args.cu_seqlens.split(",")) if args.cu_seqlens else ()

    import torch
    from paper_2506_11498_b200 import lrsa, replicas

    rank, world, local = replicas.env_rank_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    # weak scaling: every rank runs its own sequence (independent problems, no data-path collective)
    wl = replicas.rank_workload(w, rank)
    lrsa.lib()
    p = lrsa.Params.from_workload(wl, n_dense_prev=args.n_dense_prev, cu_seqlens=cu)
    host = {k: v.pin_memory() for k, v in workloads.generate(wl).items()}
    dev = {k: v.cuda(non_blocking=True) for k, v in host.items()}
    ws_sizes = lrsa.lrsa_workspace_bytes(p)
    ws = [lrsa.new_workspace(n) for n in ws_sizes]
    wsel = lrsa.lrsa_num_sel_windows(p)
    idx = torch.empty((wl.B, wl.Hkv, wsel, wl.K), dtype=torch.int32, device="cuda")
    O = torch.empty_like(dev["Q"]); LSE = torch.empty(dev["Q"].shape[:3], dtype=torch.float32, device="cuda")
    dQ = torch.empty_like(dev["Q"]); dK = torch.empty_like(dev["K"]); dV = torch.empty_like(dev["V"])
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # > 126 MB L2
    stream = torch.cuda.current_stream()
    launches = [0]

    def step(timers=None, io=None):
        """One pass of the whole path on the compute stream.  `io` = (inputs dict, (O, dQ, dK, dV)) selects
        the device buffers (the end-to-end leg double-buffers them); default: the resident set."""
        d_in, (o_, dq_, dk_, dv_) = io if io is not None else (dev, (O, dQ, dK, dV))
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)] if timers is not None else None
        if ev: ev[0].record(stream)
        lrsa.lrsa_score_select(p, d_in["K"], d_in["V"], idx=idx, workspace=ws[0])
        n = lrsa.lrsa_last_launch_count()
        if ev: ev[1].record(stream)
        lrsa.lrsa_attn_fwd(p, d_in["Q"], d_in["K"], d_in["V"], idx, O=o_, LSE=LSE, workspace=ws[1])
        n += lrsa.lrsa_last_launch_count()
        if ev: ev[2].record(stream)
        lrsa.lrsa_attn_bwd(p, d_in["Q"], d_in["K"], d_in["V"], o_, d_in["dO"], LSE, idx, dQ=dq_, dK=dk_, dV=dv_,
                           workspace=ws[2])
        n += lrsa.lrsa_last_launch_count()
        if ev:
            ev[3].record(stream)
            timers.append(ev)
        launches[0] = n

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        flush.zero_()
        step()
    barrier()
    for i, s in enumerate(ws):
        st = lrsa.lrsa_workspace_status(s)
        if st != 0:
            raise SystemExit(f"workspace {i} reports {lrsa.STATUS.get(st, st)}")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    timers = []
    barrier()
    for _ in range(args.steps):
        flush.zero_()              # L2 flush between timed iterations (outside the per-step events)
        step(timers)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    t_score = [e[0].elapsed_time(e[1]) for e in timers]
    t_fwd = [e[1].elapsed_time(e[2]) for e in timers]
    t_bwd = [e[2].elapsed_time(e[3]) for e in timers]
    t_step = [e[0].elapsed_time(e[3]) for e in timers]
    total_ms = replicas.max_over_ranks(sum(t_step), dist, "cuda")
    ms_per_step = total_ms / args.steps

    # End to end through the C ABI with HOST buffers: every step copies its Q,K,V,dO from pinned host
    # memory and reads its O,dQ,dK,dV back, all inside the timed region.  The copies run on their own
    # streams over two sets of device buffers, so step i+1's upload and step i-1's download overlap step
    # i's kernels (PCIe is full duplex), the way a training loop prefetches its next batch.
    e2e = None
    if not args.no_e2e:
        names_out = ("O", "dQ", "dK", "dV")
        outs_host = {k: torch.empty_like(v, device="cpu").pin_memory() for k, v in zip(names_out, (O, dQ, dK, dV))}
        h2d = sum(v.numel() * v.element_size() for v in host.values())
        d2h = sum(v.numel() * v.element_size() for v in outs_host.values())
        sets = [(dev, (O, dQ, dK, dV)),
                ({k: torch.empty_like(v) for k, v in dev.items()}, tuple(torch.empty_like(t) for t in (O, dQ, dK, dV)))]
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def e2e_run(n):
            ev_in = [torch.cuda.Event() for _ in range(2)]      # inputs of set k uploaded
            ev_done = [torch.cuda.Event() for _ in range(2)]    # kernels on set k finished
            ev_out = [torch.cuda.Event() for _ in range(2)]     # outputs of set k downloaded
            used = [False, False]
            s_in.wait_stream(stream); s_out.wait_stream(stream)
            for i in range(n):
                k = i % 2
                d_in, d_out = sets[k]
                with torch.cuda.stream(s_in):
                    if used[k]: s_in.wait_event(ev_done[k])      # the kernels that read this set are done
                    for name in d_in:
                        d_in[name].copy_(host[name], non_blocking=True)
                    ev_in[k].record(s_in)
                stream.wait_event(ev_in[k])
                if used[k]: stream.wait_event(ev_out[k])         # the previous results of this set are on the host
                step(io=sets[k])
                ev_done[k].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[k])
                    for name, t in zip(names_out, d_out):
                        outs_host[name].copy_(t, non_blocking=True)
                    ev_out[k].record(s_out)
                used[k] = True
            stream.wait_stream(s_out)                            # the timed region ends with the last download

        e2e_run(2); barrier()
        n_e2e = max(4, min(args.steps, 10))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        e2e_run(n_e2e)
        e1.record(stream)
        barrier()
        # the host copies are the last step's device results
        last = sets[(n_e2e - 1) % 2][1]
        for name, t in zip(names_out, last):
            if not torch.equal(outs_host[name], t.cpu()):
                raise SystemExit(f"end-to-end leg: host copy of {name} differs from the device result")
        e2e_ms = replicas.max_over_ranks(e0.elapsed_time(e1) / n_e2e, dist, "cuda")
        f_fwd, f_bwd = flops(wl, args.n_dense_prev, cu)
        e2e = {"value": replicas.job_rate(f_fwd + f_bwd, world, e2e_ms * 1e-3) / 1e12, "unit": UNIT,
               "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "overlap": "uploads, kernels and downloads of consecutive steps overlap (two buffer sets, three streams)"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    f_fwd, f_bwd = flops(wl, args.n_dense_prev, cu)
    peaks = measured_peaks()
    med = statistics.median
    bwd_s, fwd_s, score_s = med(t_bwd) * 1e-3, med(t_fwd) * 1e-3, med(t_score) * 1e-3
    # Which measured peak the kernel is held to: the burst figure when the timed region is short (under a
    # second) or ran at clocks above those of the sustained measurement, else the sustained one.  Both
    # fractions are reported; time x clock makes runs at different clocks comparable.
    timed_s = ms_per_step * 1e-3 * args.steps
    sm_mhz = (clocks or {}).get("sm_mhz")
    use_burst = timed_s < 1.0 or bool(sm_mhz and peaks.get("sustained_sm_mhz") and sm_mhz > peaks["sustained_sm_mhz"])
    peak_tf = peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"]
    achieved = f_bwd / bwd_s / 1e12
    line = {
        "metric": METRIC, "value": replicas.job_rate(f_fwd + f_bwd, world, ms_per_step * 1e-3) / 1e12, "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": wl.name, "B": wl.B, "N": wl.N, "Hq": wl.Hq, "Hkv": wl.Hkv, "d": wl.d,
                   "L": wl.L, "K": wl.K, "S": wl.S, "values": wl.values, "n_dense_prev": args.n_dense_prev,
                   "cu_seqlens": list(cu) if cu else None,
                   "l2": "256 MB buffer written between timed steps (outside the per-step events)",
                   "parallelism": f"replicas x{world} (independent sequences, no collective)"},
        "tokens_per_s": world * wl.B * wl.N / (ms_per_step * 1e-3),
        "pct_of_bf16_peak": {"measured_sustained": 100 * (f_fwd + f_bwd) / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                             "measured_burst": 100 * (f_fwd + f_bwd) / (ms_per_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
                             "nominal_2250": 100 * (f_fwd + f_bwd) / (ms_per_step * 1e-3) / 1e12 / 2250.0},
        "stages_ms": {"score_select": med(t_score), "attn_fwd": med(t_fwd), "attn_bwd": med(t_bwd),
                      "score_select_min": min(t_score), "attn_fwd_min": min(t_fwd), "attn_bwd_min": min(t_bwd)},
        "stage_rates": {"fwd_tflops": f_fwd / fwd_s / 1e12, "bwd_tflops": f_bwd / bwd_s / 1e12,
                        "score_select_gbs": kv_bytes(wl) / score_s / 1e9,
                        "score_select_frac_of_hbm": kv_bytes(wl) / score_s / 1e9 / peaks["hbm_gbs"]},
        # achieved = effective backward FLOPs (10*d per unmasked pair) / the backward call's CUDA-event time
        # (dK/dV kernel + dQ kernel + ~2 % helpers).  traffic: DRAM bytes of those two kernels in one launch
        # each from an ncu capture; null while the kernels are newer than the last capture.
        "roofline": {"kernel": "lrsa_attn_bwd (lrsa_bwd_dkv_kernel + lrsa_bwd_dq_kernel)", "bound": "tensor",
                     "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved / peak_tf,
                     "frac_burst": achieved / peaks["bf16_tflops"],
                     "frac_sustained": achieved / peaks["bf16_tflops_sustained"],
                     "traffic": BWD_DRAM_BYTES.get(wl.name) if not cu else None,
                     "ms_x_sm_mhz": None if not sm_mhz else med(t_bwd) * sm_mhz,
                     "peak_source": f"{peaks['source']} {'burst' if use_burst else 'sustained'} bf16 "
                                    f"(timed region {timed_s:.2f} s at {sm_mhz} MHz)"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches[0] * args.steps,
    }
    if not args.no_decode and world == 1 and not cu and args.n_dense_prev == 1:
        line["decode"] = decode_leg(lrsa, torch, wl, p, dev, flush, peaks)
    if not args.no_cpu_baseline and world == 1:
        s = oracle_sample(w, n_chunks=3, host={k: v for k, v in host.items()} if wl.seed == w.seed else None)
        line["cpu_baseline"] = {"value": s["tflops"], "unit": UNIT, "cores": s["cores"], "kind": "oracle",
                                "sample": s["sample"]}
        if not cu:   # packed batches are covered by the tests
            line["parity_sample"] = parity_sample(wl, host, (O, dQ), idx, args.n_dense_prev)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
