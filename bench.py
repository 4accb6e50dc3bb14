#!/usr/bin/env python
"""Benchmark of the batched LQR solve (one "step" = one ttc_lqr_solve over the whole workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--method auto|riccati|scan]
    python bench.py --impl reference ...      # the float64 CPU oracle on the host cores

Prints ONE JSON line.  `value` is instances/s with the inputs resident in HBM, timed with CUDA
events on the launching stream (max over ranks).  `e2e` is the same metric through
ttc_lqr_solve_host with pinned host buffers, copies inside the timed region.  `roofline`
describes the dominant kernel; `cpu_baseline` is the oracle, as it stands, on a bounded sample.
With N > 1 (torchrun) every rank solves its own copy of the workload (instances are independent:
weak scaling, no collective on the data path).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_09221_b200 import sharding, workloads  # noqa: E402

SM_COUNT = 148
FP32_LANES_PER_SM = 128
TF32_TO_BF16_RATIO = 0.5     # nominal dense tensor ratio tf32 : bf16 on B200 (1.1 : 2.25 PFLOP/s)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d["bf16_tflops_sustained"], sm_max_mhz=d.get("sm_max_mhz", 1965.0),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0,
                source="fallback")


def algorithmic_counts(c):
    """Per-instance algorithmic flops (symmetry-exploiting Riccati count) and HBM bytes
    (inputs once + requested fp32 outputs once)."""
    n, m, H = c["n"], c["m"], c["H"]
    flops = (3 * n**3 + 5 * n * n * m + 3 * n * m * m + m**3 / 3.0 + 2 * n * n + 4 * n * m) * H
    esz = 2 if c["q_dtype"] == "bf16" else 4
    bytes_in = (n * n + n) * esz
    if c.get("tv"):                  # per-token Q_t for every step plus the terminal weight; head operands are shared
        bytes_in = ((H + 1) * n * n + n) * esz
    if c["first_only"]:
        bytes_out = 4 * (n * n + m)
    else:
        bytes_out = 4 * (H * m * n + (H + 1) * n * n + (H + 1) * n + H * m)
    return flops, bytes_in, bytes_out


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self._stop = threading.Event()
        self._t = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 8:
                    self.rows.append(parts)
            except Exception:
                pass
            self._stop.wait(0.1)

    def start(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()

    def stop(self):
        self._stop.set()
        if self._t:
            self._t.join(timeout=6)
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(self.rows)}


def oracle_sample(w, count):
    """Stratified sample of instance indices covering every (seq, head)."""
    S, Hd, T = w["batch"]
    per = max(1, count // (S * Hd))
    toks = np.unique(np.linspace(0, T - 1, per).astype(np.int64))
    idx = (np.arange(S * Hd)[:, None] * T + toks[None, :]).reshape(-1)
    return idx


def time_oracle(w, idx, first_only):
    from tests import parity_util as pu
    t0 = time.perf_counter()
    ref = (pu.run_oracle_tv if w.get("tv") else pu.run_oracle)(w, idx=idx, first_only=first_only)
    dt = time.perf_counter() - t0
    return ref, dt


def run_reference(args, cid, tv_key=None):
    """--impl reference: the float64 oracle on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    c = workloads.TV_CONFIGS[tv_key] if tv_key else workloads.CONFIGS[cid]
    S, Hd, T = c["batch"]
    tok = max(1, min(T, args.ref_instances // (S * Hd)))
    n_inst = S * Hd * tok
    from oracle import lqr_oracle as orc
    want = ("P", "u") if c["first_only"] else ("K", "P", "x", "u")
    if tv_key:
        w = workloads.make_tv_workload(tv_key, device="cpu", batch=(S, Hd, tok))
        d = {k: w[k].to(torch.float64).numpy() for k in ("A", "B", "Q", "R", "Qf", "x0")}
        solve = lambda: orc.solve_batch_tv(d["A"], d["B"], d["Q"], d["R"], d["Qf"], d["x0"], c["H"], (S, Hd, tok),
                                           tv=c["tv"], first_only=c["first_only"], want=want)
    else:
        from paper_2603_09221_b200.workloads import to_float64_numpy
        d = to_float64_numpy(workloads.make_workload(cid, device="cpu", batch=(S, Hd, tok)))
        solve = lambda: orc.solve_batch(d["A"], d["B"], d["Q"], d["R"], d["x0"], c["H"], batch=(S, Hd, tok),
                                        first_only=c["first_only"], want=want)
    times, threads = [], 0
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        out = solve()
        dt = time.perf_counter() - t0
        threads = out["threads"]
        if it >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = n_inst / (ms * 1e-3)
    line = {"impl": "reference", "metric": "lqr_instances_per_sec", "value": val, "unit": "instances/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": c["name"], "n": c["n"], "m": c["m"], "H": c["H"],
                       "instances_per_step": n_inst, "note": "bounded sample of the workload per step"},
            "cpu_baseline": {"value": val, "unit": "instances/s", "cores": threads, "kind": "oracle",
                             "sample": "%d instances (%dx%dx%d tokens) per step" % (n_inst, S, Hd, tok)},
            "e2e": {"value": val, "unit": "instances/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


GRAD_NAMES = ("dA", "dB", "dQ", "dQf", "dR", "dx0", "u0")


def grad_oracle(w, g, idx, H):
    """Thm 3.2 gradients of the sampled instances by the float64 oracle (one instance at a time)."""
    from oracle import lqr_grad as og
    S, Hd, T = w["batch"]
    f64 = lambda t: t.to(torch.float64).cpu().numpy()
    t0 = time.perf_counter()
    refs = []
    def head_or_token(t, i):                                 # A, B, R: [1, Hd, 1, ...] per head or [S, Hd, T, ...] per token
        if t.shape[2] == 1:
            return t[0, (int(i) // T) % Hd, 0]
        return t.reshape((-1,) + t.shape[3:])[i]

    for i in idx:
        refs.append(og.grad(f64(head_or_token(w["A"], i)), f64(head_or_token(w["B"], i)), f64(w["Q"].reshape((-1,) + w["Q"].shape[3:])[i]),
                            f64(head_or_token(w["R"], i)), f64(w["Qf"].reshape((-1,) + w["Qf"].shape[3:])[i]),
                            f64(w["x0"].reshape(-1, w["x0"].shape[-1])[i]), f64(g[i]), H))
    ref = {k: np.stack([r[k] for r in refs]) for k in GRAD_NAMES}
    return ref, time.perf_counter() - t0


def run_grad(args):
    """--workload grad16: one step = one ttc_lqr_grad over the whole workload (backward pass, both rollouts and
    co-state sequences, outer products), every gradient written."""
    key = args.workload
    c = dict(workloads.TV_CONFIGS[key])
    if args.horizon > 0:
        c["H"] = args.horizon
        c["name"] += "_T%d" % args.horizon
    if args.batch:
        c["batch"] = tuple(int(v) for v in args.batch.split("x"))
        c["name"] += "_batch" + args.batch
    rank = int(os.environ.get("RANK", "0"))
    n, m, H = c["n"], c["m"], c["H"]
    if args.impl == "reference":
        if rank != 0:
            return
        S, Hd, Tk = c["batch"]
        cnt = max(1, min(S * Hd * Tk, args.ref_instances // 8))
        w = workloads.make_tv_workload(key, device="cpu", batch=(1, Hd, max(1, cnt // Hd)), horizon=H)
        Nw = int(np.prod(w["batch"]))
        g = torch.randn((Nw, m), generator=torch.Generator().manual_seed(7))
        times = []
        for it in range(args.warmup + args.steps):
            _, dt = grad_oracle(w, g, range(Nw), H)
            if it >= args.warmup:
                times.append(dt)
        ms = 1e3 * sum(times) / len(times)
        val = Nw / (ms * 1e-3)
        print(json.dumps({"impl": "reference", "metric": "lqr_instances_per_sec", "value": val, "unit": "instances/s",
                          "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic",
                          "config": {"workload": c["name"], "n": n, "m": m, "H": H, "instances_per_step": Nw,
                                     "note": "bounded sample of the workload per step"},
                          "cpu_baseline": {"value": val, "unit": "instances/s", "cores": 1, "kind": "oracle",
                                           "sample": "%d instances per step, one at a time" % Nw},
                          "e2e": {"value": val, "unit": "instances/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}))
        return
    args.warmup = max(args.warmup, 3)
    from paper_2603_09221_b200 import lqr
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the solver has no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = world > 1
    if dist:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = measured_peaks()
    if args.tokens > 0:
        c["batch"] = (c["batch"][0], c["batch"][1], args.tokens)
        c["name"] += "_tokens%d" % args.tokens
    w = workloads.make_tv_workload(key, device=dev, batch=c["batch"], seed=sharding.rank_seed(100, rank), horizon=H)
    N = int(np.prod(c["batch"]))
    if args.per_token:
        # the contextualised layer's situation: every token its own A_t, B_t, R_t (here copies of the head's, which
        # costs the same traffic and arithmetic as distinct ones)
        for k in ("A", "B", "R"):
            w[k] = w[k].expand(tuple(c["batch"]) + w[k].shape[3:]).contiguous()
        c["name"] += "_per_token"
    gen = torch.Generator(device=dev)
    gen.manual_seed(sharding.rank_seed(300, rank))
    g = torch.randn((N, m), generator=gen, device=dev)
    solver = lqr.LqrSolver(n, m, H, c["batch"], device=local)
    shp = dict(dA=(N, H, n, n), dB=(N, H, n, m), dQ=(N, H, n, n), dQf=(N, n, n), dR=(N, H, m, m), dx0=(N, n), u0=(N, m))
    out = {k: torch.empty(v, device=dev) for k, v in shp.items()}
    out["info"] = torch.empty((N,), dtype=torch.int32, device=dev)

    def step():
        solver.grad(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], g, H, tv=c["tv"], **out)

    def barrier():
        if dist:
            td.barrier()
        torch.cuda.synchronize(dev)

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    evs[0].record()
    for i in range(args.steps):
        step()
        evs[i + 1].record()
    barrier()
    launches = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES) - launches0
    clocks = sampler.stop() if rank == 0 else None
    per_step = [evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps)]
    value, ms_per_step, _ = sharding.aggregate_throughput(N, evs[0].elapsed_time(evs[-1]) / args.steps, device=dev)
    if rank != 0:
        if dist:
            td.destroy_process_group()
        return
    # algorithmic bytes: Q_t, Q_f, x_0, g in (the per-head A_t, B_t, R_t are negligible); every gradient, u_0, info out
    bin_i = 4 * (H * n * n + n * n + n + m) + (4 * H * (n * n + n * m + m * m) if args.per_token else 0)
    bout_i = 4 * (H * (2 * n * n + n * m + m * m) + n * n + n + m + 1)
    kernel_ms = statistics.median(per_step)
    ach = N * (bin_i + bout_i) / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "traffic": None, "kernel": "whole step: backward pass + grad_vectors + grad_outer (3 launches)",
                "kernel_ms": kernel_ms, "peak_note": "copy bandwidth, of %s" % peaks["source"],
                "algorithmic_bytes_per_launch": N * (bin_i + bout_i)}
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        idx = np.unique(np.linspace(0, N - 1, max(8, args.cpu_sample // 8)).astype(np.int64))
        ref, dt = grad_oracle(w, g, idx, H)
        from tests import parity_util as pu
        sel = torch.as_tensor(idx)
        # per instance, relative to the largest entry of that gradient over the horizon; Q_f is the last member of the
        # state-cost sequence and is measured with it (x_H decays with the horizon, and with it dQf's own scale)
        got = {k: out[k].cpu()[sel].reshape(len(idx), -1).numpy() for k in GRAD_NAMES}
        exp = {k: ref[k].reshape(len(idx), -1) for k in GRAD_NAMES}
        got["dQ"] = np.concatenate([got["dQ"], got.pop("dQf")], axis=1)
        exp["dQ"] = np.concatenate([exp["dQ"], exp.pop("dQf")], axis=1)
        errs = {("dQ+dQf" if k == "dQ" else k): pu.block_rel_err(got[k], exp[k], 1, per_block=False) for k in got}
        assert all(v <= c["tol"] for v in errs.values()), errs
        assert int(out["info"].abs().max()) == 0
        cpu = {"value": len(idx) / dt, "unit": "instances/s", "cores": 1, "kind": "oracle",
               "sample": "%d instances spread over the workload, one at a time" % len(idx),
               "seconds": dt, "parity_max_rel_err": errs, "speedup_gpu_over_cpu": value / (len(idx) / dt)}
    print(json.dumps({"metric": "lqr_instances_per_sec", "value": value, "unit": "instances/s", "n_gpus": world,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": c["name"], "n": n, "m": m, "H": H, "instances": N, "batch": list(c["batch"]),
                                 "time_varying": list(c["tv"]), "outputs": list(GRAD_NAMES) + ["info"],
                                 "l2": "inputs+outputs per step exceed L2 (%.2f GB)" % (N * (bin_i + bout_i) / 1e9)},
                      "roofline": roofline, "cpu_baseline": cpu, "e2e": None,
                      "e2e_note": "gradients stay on the device for the layers below; no host-buffer entry point",
                      "gpu_launches": int(launches), "launches_per_step": launches / args.steps, "clocks": clocks,
                      "ms_per_step_percentiles": {"p20": float(np.percentile(per_step, 20)),
                                                  "p50": float(np.percentile(per_step, 50)),
                                                  "p80": float(np.percentile(per_step, 80))}}))
    solver.close()
    if dist:
        td.destroy_process_group()


def layer_counts(c):
    """Per-instance algorithmic flops and HBM bytes of the contextualised layer solve: per step P Bbar (2 n^3),
    Bbar'V (n^3, S symmetric), Cholesky (n^3 / 3), L^{-1}Y (n^3), Z'Z (n^3, symmetric); Y = G Bbar'P A_t is the
    transpose of P Bbar scaled on both sides (A_t diagonal) and costs no contraction; per instance the synthesis of
    Bbar, Qbar, Q_T (6 r n^2).  Bytes: coefficient vectors in, u_1* and P_0 out."""
    n, r, T = c["n"], c["r"], c["T"]
    flops = (5.0 + 1.0 / 3.0) * n**3 * T + 6.0 * r * n * n
    return flops, 4 * (6 * n + 3 * r), 4 * (n + n * n)


def layer_oracle(w, idx, T):
    from oracle import ttc_layer as lay
    sel = lambda k: w[k][torch.as_tensor(idx, device=w[k].device)].to(torch.float64).cpu().numpy()
    f64 = lambda k: w[k].to(torch.float64).cpu().numpy()
    t0 = time.perf_counter()
    ref = lay.solve_batch(sel("s_a"), sel("s_gamma_a"), sel("s_gamma_b"), sel("s_gamma_q"), sel("s_b"), sel("s_q"),
                          sel("s_qf"), sel("r_inv"), sel("h0"), f64("B_basis"), f64("Q_basis"), T)
    return ref, time.perf_counter() - t0


def run_layer(args):
    """--workload layer16 / layer32: one step = one ttc_lqr_solve_layer over the whole workload."""
    key = args.workload
    c = dict(workloads.LAYER_CONFIGS[key])
    if args.horizon > 0:
        c["T"] = args.horizon
        c["name"] += "_T%d" % args.horizon
    if args.batch:
        c["batch"] = tuple(int(v) for v in args.batch.split("x"))
        c["name"] += "_batch" + args.batch
    rank = int(os.environ.get("RANK", "0"))
    if args.impl == "reference":
        if rank != 0:
            return
        S, Hd, Tk = c["batch"]
        tok = max(1, min(Tk, args.ref_instances // (S * Hd)))
        w = workloads.make_layer_workload(key, device="cpu", batch=(S, Hd, tok))
        idx = np.arange(w["N"])
        times, threads = [], 0
        for it in range(args.warmup + args.steps):
            ref, dt = layer_oracle(w, idx, c["T"])
            threads = int(ref["threads"])
            if it >= args.warmup:
                times.append(dt)
        ms = 1e3 * sum(times) / len(times)
        val = w["N"] / (ms * 1e-3)
        print(json.dumps({"impl": "reference", "metric": "lqr_instances_per_sec", "value": val, "unit": "instances/s",
                          "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                          "data": "synthetic",
                          "config": {"workload": c["name"], "n": c["n"], "r": c["r"], "T": c["T"],
                                     "instances_per_step": w["N"], "note": "bounded sample of the workload per step"},
                          "cpu_baseline": {"value": val, "unit": "instances/s", "cores": threads, "kind": "oracle",
                                           "sample": "%d instances per step (parameter synthesis in numpy + C recursion)" % w["N"]},
                          "e2e": {"value": val, "unit": "instances/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}))
        return
    args.warmup = max(args.warmup, 3)
    from paper_2603_09221_b200 import lqr
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the solver has no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = world > 1
    if dist:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = measured_peaks()
    if args.tokens > 0:
        c["batch"] = (c["batch"][0], c["batch"][1], args.tokens)
        c["name"] += "_tokens%d" % args.tokens
    w = workloads.make_layer_workload(key, device=dev, batch=c["batch"], seed=sharding.rank_seed(200, rank))
    n, r, T, N = c["n"], c["r"], c["T"], w["N"]
    solver = lqr.LqrSolver(n, n, T, c["batch"], device=local)
    u1 = torch.empty((N, n), device=dev)
    P0 = torch.empty((N, n, n), device=dev)
    info = torch.empty((N,), dtype=torch.int32, device=dev)
    ins = [w[k] for k in workloads.LAYER_KEYS]

    baseline = args.method == "sigma"      # the row-normalised reverse symplectic product instead of the recursion
    if baseline:
        c["name"] += "_sigma_baseline"
        args.no_e2e = True

    gradient = args.grad                   # ttc_lqr_layer_grad: backward of the layer output w.r.t. every coefficient
    if gradient:
        c["name"] += "_grad"
        args.no_e2e = True
        gen = torch.Generator(device=dev)
        gen.manual_seed(sharding.rank_seed(400, rank))
        gout = torch.randn((N, n), generator=gen, device=dev)
        grads = {k: torch.empty_like(w[k]) for k in lqr.LAYER_GRAD_KEYS}

    def step():
        if gradient:
            solver.layer_grad(*ins, T, gout, grads, u1=u1, info=info)
        elif baseline:
            solver.solve_layer_sigma_baseline(*ins, T, u1=u1, P0=P0, info=info)
        else:
            solver.solve_layer(*ins, T, u1=u1, P0=P0, info=info)

    def barrier():
        if dist:
            td.barrier()
        torch.cuda.synchronize(dev)

    # the working set (a few MB) fits L2: flush it between timed steps by writing a buffer larger than L2
    flush = torch.empty(192 * 1024 * 1024, dtype=torch.uint8, device=dev)
    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    for i in range(args.steps):
        flush.fill_(i & 255)
        e0[i].record()
        step()
        e1[i].record()
    barrier()
    launches = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES) - launches0
    clocks = sampler.stop() if rank == 0 else None
    per_step = [e0[i].elapsed_time(e1[i]) for i in range(args.steps)]
    value, ms_per_step, _ = sharding.aggregate_throughput(N, sum(per_step) / len(per_step), device=dev)

    e2e = None
    if not args.no_e2e:
        # end to end through ttc_lqr_solve_layer_host: coefficient vectors in pinned host memory, u_1*, P_0, info back
        hin = [t.cpu().pin_memory() for t in ins]
        hu, hP = torch.empty((N, n)).pin_memory(), torch.empty((N, n, n)).pin_memory()
        hinfo = torch.empty((N,), dtype=torch.int32).pin_memory()
        h2d = sum(t.numel() * t.element_size() for t in hin)
        d2h = hu.numel() * 4 + hP.numel() * 4 + hinfo.numel() * 4

        def host_step():
            solver.solve_layer_host(*hin, T, u1=hu, P0=hP, info=hinfo)

        host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
        barrier()
        e2e_ms = 1e3 * (time.perf_counter() - t0) / args.e2e_steps
        e2e_value, e2e_ms_max, _ = sharding.aggregate_throughput(N, e2e_ms, device=dev)
        e2e = {"value": e2e_value, "unit": "instances/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "ms_per_step": e2e_ms_max}
    if rank != 0:
        if dist:
            td.destroy_process_group()
        return
    flops_i, bin_i, bout_i = layer_counts(c)
    kernel_ms = statistics.median(per_step)
    fp32_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    ach = N * flops_i / (kernel_ms * 1e-3) / 1e12
    roofline = {"bound": "alu", "achieved": ach, "peak": fp32_peak, "unit": "TFLOP/s", "frac": ach / fp32_peak,
                "traffic": None, "kernel": "ttc_layer", "kernel_ms": kernel_ms,
                "peak_note": "148 SMs x 128 FP32 lanes x 2 x %.0f MHz (derived)" % peaks["sm_max_mhz"],
                "algorithmic_flops_per_launch": N * flops_i, "algorithmic_bytes_per_launch": N * (bin_i + bout_i),
                "hbm_frac": (N * (bin_i + bout_i) / (kernel_ms * 1e-3) / 1e9) / peaks["hbm_gbs"]}
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        idx = np.unique(np.linspace(0, N - 1, args.cpu_sample if not gradient else max(8, args.cpu_sample // 64)).astype(np.int64))
        from tests import parity_util as pu
        sel = torch.as_tensor(idx)
        if gradient:                       # per-instance gradients against the float64 gradient oracle, one instance at a time
            from oracle import ttc_layer_grad as og
            f64 = lambda t: t.to(torch.float64).cpu().numpy()
            t0 = time.perf_counter()
            refs = [og.grad(*(f64(w[k][i]) for k in workloads.LAYER_KEYS[:9]), f64(w["B_basis"]), f64(w["Q_basis"]), T, f64(gout[i]))
                    for i in idx]
            dt = time.perf_counter() - t0
            ref = {"threads": 1}
            errs = {}
            for k in lqr.LAYER_GRAD_KEYS[:9]:
                got = grads[k].cpu()[sel].double().numpy()
                exp = np.stack([r_[k] for r_ in refs])
                errs[k] = float((np.abs(got - exp).max(axis=1) / np.maximum(np.abs(exp).max(axis=1), 1e-30)).max())
            assert all(v <= c["tol"] for v in errs.values()), errs
            assert int(info.abs().max()) == 0
        elif baseline:
            ref, dt = layer_oracle(w, idx, T)                       # a baseline whose float32 error grows with the horizon: reported, not gated
            g_u, g_P = u1.cpu()[sel].double().numpy(), P0.cpu()[sel].double().numpy().reshape(len(idx), -1)
            eu = np.abs(g_u - ref["u1"]).max(axis=1) / np.abs(ref["u1"]).max(axis=1)
            eP = np.abs(g_P - ref["P0"].reshape(len(idx), -1)).max(axis=1) / np.abs(ref["P0"]).reshape(len(idx), -1).max(axis=1)
            errs = {"u1_median": float(np.nanmedian(eu)), "u1_p90": float(np.nanpercentile(eu, 90)),
                    "P0_median": float(np.nanmedian(eP)), "P0_p90": float(np.nanpercentile(eP, 90)),
                    "singular_Y1": int((info.cpu()[sel] != 0).sum())}
        else:
            ref, dt = layer_oracle(w, idx, T)
            errs = {"P0": pu.block_rel_err(P0.cpu()[sel].numpy(), ref["P0"], 2),
                    "u1": pu.block_rel_err(u1.cpu()[sel].numpy(), ref["u1"], 1)}
            assert all(v <= c["tol"] for v in errs.values()), errs
            assert int(info.abs().max()) == 0
        cpu = {"value": len(idx) / dt, "unit": "instances/s", "cores": int(ref["threads"]), "kind": "oracle",
               "sample": "%d instances spread over the workload (parameter synthesis in numpy + C recursion)" % len(idx),
               "seconds": dt, "parity_max_rel_err": errs, "speedup_gpu_over_cpu": value / (len(idx) / dt)}
    print(json.dumps({"metric": "lqr_instances_per_sec", "value": value, "unit": "instances/s", "n_gpus": world,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                      "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                      "config": {"workload": c["name"], "n": n, "r": r, "T": T, "instances": N, "batch": list(c["batch"]),
                                 "outputs": ["u1", "P0", "info"], "kernel": "sigma_product (baseline)" if baseline else "ttc_layer",
                                 "l2": "working set fits L2: a 192 MB buffer is written between timed steps"},
                      "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
                      "launches_per_step": launches / args.steps, "clocks": clocks}))
    solver.close()
    if dist:
        td.destroy_process_group()


def measure_run_peaks(local, dev):
    """FP32 FMA and TF32 tensor peaks measured in this run on this device (the denominators of the "alu" and
    "tensor" roofline fractions): an FMA-chain micro-kernel of the library, and an 8192^3 float32 matmul with TF32
    tensor cores allowed (cuBLAS through torch), best of 5 (burst) and back to back for about a second (sustained)."""
    from paper_2603_09221_b200 import lqr
    sampler = ClockSampler(local)
    sampler.start()
    scalar, packed = lqr.measure_fp32_peak(local)
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        M = 8192
        a = torch.randn((M, M), device=dev)
        b = torch.randn((M, M), device=dev)
        c = torch.empty((M, M), device=dev)
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize(dev)
        flops = 2.0 * M ** 3
        burst = 0.0
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch.matmul(a, b, out=c)
            e1.record()
            torch.cuda.synchronize(dev)
            burst = max(burst, flops / (e0.elapsed_time(e1) * 1e-3) / 1e12)
        reps = max(8, int(1.0 / (flops / (burst * 1e12))))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record()
        torch.cuda.synchronize(dev)
        sustained = reps * flops / (e0.elapsed_time(e1) * 1e-3) / 1e12
        del a, b, c
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old
    clocks = sampler.stop()
    return {"fp32_tflops": max(scalar, packed), "fp32_tflops_scalar_fma": scalar, "fp32_tflops_packed_fma": packed,
            "tf32_tflops": burst, "tf32_tflops_sustained": sustained,
            "how": "FMA-chain micro-kernel (ttc_lqr_measure_fp32_peak, best of 5); torch.matmul fp32 8192^3 with TF32 "
                   "allowed, best of 5 and %d back to back" % reps,
            "clocks": clocks}


def run_solve(args, workload, method_name, ctx, light=False):
    """One workload of ttc_lqr_solve / ttc_lqr_solve_tv through the C ABI: warm-up, timed steps (CUDA events), end to
    end through the host-buffer entry, roofline of the dominant kernel, parity and CPU baseline on a sample.
    Returns the JSON line as a dict on rank 0 (None on the other ranks).  `light`: a short side measurement (fewer
    steps, no end-to-end leg)."""
    from paper_2603_09221_b200 import lqr
    dist, world, rank, local, dev, peaks, run_peaks = (ctx[k] for k in ("dist", "world", "rank", "local", "dev", "peaks", "run_peaks"))
    if dist:
        import torch.distributed as td
    tv_key = workload if workload in workloads.TV_CONFIGS else None
    cid = None if tv_key else int(workload.replace("cfg", ""))
    steps = 5 if light else args.steps
    warmup = 3 if light else args.warmup
    no_e2e = args.no_e2e or light or bool(tv_key)     # the host-buffer entry point covers the time-invariant solve only

    c = dict(workloads.TV_CONFIGS[tv_key] if tv_key else workloads.CONFIGS[cid])
    if args.tokens > 0:
        c["batch"] = (c["batch"][0], c["batch"][1], args.tokens)
        c["name"] += "_tokens%d" % args.tokens
    if tv_key:
        w = workloads.make_tv_workload(tv_key, device=dev, batch=c["batch"], seed=sharding.rank_seed(100, rank))
    else:
        w = workloads.make_workload(cid, device=dev, batch=c["batch"], seed=sharding.rank_seed(cid, rank))
    n, m, H = c["n"], c["m"], c["H"]
    N = int(np.prod(c["batch"]))
    first = c["first_only"]
    method = {"auto": lqr.TTC_AUTO, "riccati": lqr.TTC_RICCATI, "scan": lqr.TTC_SCAN}[method_name]
    math = {"auto": lqr.TTC_MATH_AUTO, "fp32": lqr.TTC_MATH_FP32, "tf32": lqr.TTC_MATH_TF32}[args.math]
    solver = lqr.LqrSolver(n, m, H, c["batch"], device=local, method=method, math=math)
    want = ("P", "u", "info") if first else ("K", "P", "x", "u", "info")
    obf = args.out_dtype == "bf16" and not tv_key and not light
    lowrank = args.lowrank_q and "U" in w and not light
    out = lqr.alloc_outputs(n, m, H, N, dev, first_only=first, want=want, dtype=torch.bfloat16 if obf else torch.float32)
    flags = (lqr.TTC_OUT_FIRST_ONLY if first else 0) | (lqr.TTC_OUT_BF16 if obf else 0)
    if lowrank:
        no_e2e = True                      # the host-buffer entry point takes dense Q
    if obf or lowrank:
        c["name"] += ("_outbf16" if obf else "") + ("_lowrankq" if lowrank else "")

    def step():
        if lowrank:
            solver.solve_lowrank_q(w["A"], w["B"], w["U"], w["d"], w["q_scale"], w["R"], w["x0"], H, K=out.get("K"),
                                   P=out.get("P"), x=out.get("x"), u=out.get("u"), info=out.get("info"), flags=flags)
            return
        if tv_key:
            solver.solve_tv(w["A"], w["B"], w["Q"], w["R"], w["Qf"], w["x0"], H, tv=c["tv"], K=out.get("K"),
                            P=out.get("P"), x=out.get("x"), u=out.get("u"), info=out.get("info"), flags=flags)
            return
        solver.solve(w["A"], w["B"], w["Q"], w["R"], w["x0"], H, K=out.get("K"), P=out.get("P"), x=out.get("x"),
                     u=out.get("u"), info=out.get("info"), flags=flags)

    def barrier():
        if dist:
            td.barrier()
        torch.cuda.synchronize(dev)

    flops_i, bin_i, bout_i = algorithmic_counts(c)
    if obf:
        bout_i = bout_i // 2               # bfloat16 outputs
    if lowrank:
        bin_i = (n * 8 + n + n) * (2 if c["q_dtype"] == "bf16" else 4)      # U, d, x0
    alg_bytes = N * (bin_i + bout_i)
    alg_flops = N * flops_i
    # inputs + outputs of the large configurations exceed L2 several times over; the small ones fit, so a buffer
    # larger than L2 is written between their timed steps
    flush = torch.empty(192 * 1024 * 1024, dtype=torch.uint8, device=dev) if alg_bytes <= 256e6 else None
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES)
    e0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    e1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    barrier()
    for i in range(steps):
        if flush is not None:
            flush.fill_(i & 255)
        e0[i].record()
        step()
        e1[i].record()
    barrier()
    launches = solver.query(lqr.TTC_QUERY_TOTAL_LAUNCHES) - launches0
    clocks = sampler.stop() if rank == 0 else None
    per_step = [e0[i].elapsed_time(e1[i]) for i in range(steps)]
    kernel_id = solver.query(lqr.TTC_QUERY_LAST_KERNEL)
    value, ms_per_step, _ = sharding.aggregate_throughput(N, sum(per_step) / steps, device=dev)
    del flush

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed)
    e2e = None
    if not no_e2e:
        hin = {k: w[k].cpu().pin_memory() for k in ("A", "B", "Q", "R", "x0")}
        hout = lqr.alloc_outputs(n, m, H, N, "cpu", first_only=first, want=want, pin=True,
                                 dtype=torch.bfloat16 if obf else torch.float32)
        h2d = sum(v.numel() * v.element_size() for v in hin.values())
        d2h = sum(v.numel() * v.element_size() for v in hout.values())

        def host_step():
            solver.solve_host(hin["A"], hin["B"], hin["Q"], hin["R"], hin["x0"], H, K=hout.get("K"), P=hout.get("P"),
                              x=hout.get("x"), u=hout.get("u"), info=hout.get("info"), flags=flags)

        host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            host_step()
        barrier()
        e2e_ms = 1e3 * (time.perf_counter() - t0) / args.e2e_steps
        e2e_value, e2e_ms_max, _ = sharding.aggregate_throughput(N, e2e_ms, device=dev)
        e2e = {"value": e2e_value, "unit": "instances/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms_max}
        del hin, hout

    if rank != 0:
        solver.close()
        return None

    # ---- roofline of the dominant kernel (one launch per step does the whole backward pass)
    kname = lqr.KERNEL_NAMES.get(kernel_id, str(kernel_id))
    launches_per_step = launches / steps
    kernel_ms = statistics.median(per_step)       # dominant kernel ~ the whole step (events per step)
    t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
    fp32_derived = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    tf32_derived = peaks["bf16_tflops_sustained"] * TF32_TO_BF16_RATIO
    fp32_peak = run_peaks["fp32_tflops"] if run_peaks else fp32_derived
    tf32_peak = run_peaks["tf32_tflops_sustained"] if run_peaks else tf32_derived
    extra = {}
    if kname == "riccati_umma" and alg_flops / (tf32_peak * 1e12) >= t_hbm:
        bound, peak, unit, ach = "tensor", tf32_peak, "TFLOP/s", alg_flops / (kernel_ms * 1e-3) / 1e12
        peak_note = ("tf32 matmul (cuBLAS via torch) measured in this run, sustained" if run_peaks else
                     "tf32 = measured sustained bf16 x 0.5 (nominal ratio), of %s" % peaks["source"])
        extra = {"frac_of_half_bf16_sustained": ach / tf32_derived, "half_bf16_sustained_tflops": tf32_derived}
    elif kname == "riccati_umma":          # every K_t, P_t written: the bytes take longer than the flops at the tensor peak
        bound, peak, unit, ach = "hbm", peaks["hbm_gbs"], "GB/s", alg_bytes / (kernel_ms * 1e-3) / 1e9
        peak_note = "copy bandwidth, of %s (the tensor-core time at the measured tf32 peak is shorter)" % peaks["source"]
        extra = {"tensor_frac": (alg_flops / (kernel_ms * 1e-3) / 1e12) / tf32_peak, "tf32_peak_tflops": tf32_peak}
    else:
        t_alu = alg_flops / (fp32_peak * 1e12)
        if t_hbm >= t_alu:
            bound, peak, unit, ach = "hbm", peaks["hbm_gbs"], "GB/s", alg_bytes / (kernel_ms * 1e-3) / 1e9
            peak_note = "copy bandwidth, of %s" % peaks["source"]
        else:
            bound, peak, unit, ach = "alu", fp32_peak, "TFLOP/s", alg_flops / (kernel_ms * 1e-3) / 1e12
            peak_note = ("FMA-chain micro-kernel measured in this run" if run_peaks else
                         "148 SMs x 128 FP32 lanes x 2 x %.0f MHz (derived)" % peaks["sm_max_mhz"])
            extra = {"frac_of_derived_peak": ach / fp32_derived, "derived_peak_tflops": fp32_derived}
    roofline = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak, "traffic": None,
                "kernel": kname, "kernel_ms": kernel_ms, "peak_note": peak_note,
                "algorithmic_flops_per_launch": alg_flops, "algorithmic_bytes_per_launch": alg_bytes,
                "hbm_frac": (alg_bytes / (kernel_ms * 1e-3) / 1e9) / peaks["hbm_gbs"]}
    roofline.update(extra)
    if method_name == "scan":
        # the scan executes its own flop count: per doubling round one squaring of the element and the applications
        # of the round; reported beside the Riccati-equivalent figure above
        roofline["nominal_B_T_d3_flops"] = float(N) * H * n ** 3
    traffic_path = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(traffic_path):
        with open(traffic_path) as f:
            tr = json.load(f).get("%s/%s" % (c["name"], kname))
        if tr:
            roofline["traffic"] = tr["dram_bytes_per_instance"] * N
            roofline["traffic_note"] = tr.get("note")

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        # parity of the timed configuration on a stratified sample (every sequence and head), oracle timed on it
        idx = oracle_sample(w, args.cpu_sample)
        from tests import parity_util as pu
        if lowrank:                        # the oracle gets the dense Q that the factors describe, formed in float64
            from oracle import lqr_oracle as orc
            A_, B_, _, R_, x0_ = pu.gather_inputs(w, idx)
            sel = torch.as_tensor(idx, device=dev)
            U_ = w["U"].reshape(N, n, 8)[sel].double().cpu().numpy()
            d_ = w["d"].reshape(N, n)[sel].double().cpu().numpy()
            Q_ = w["q_scale"] * U_ @ np.swapaxes(U_, 1, 2) + d_[:, :, None] * np.eye(n)
            t0 = time.perf_counter()
            ref = orc.solve_batch(A_, B_, Q_, R_, x0_, H, batch=(len(idx),), first_only=first)
            dt = time.perf_counter() - t0
        else:
            ref, dt = time_oracle(w, idx, first)
        got = {k: (v.float() if v.dtype == torch.bfloat16 else v) for k, v in out.items()}
        errs = pu.compare(got, ref, idx, c["tol"] + (2.0 ** -8 if obf else 0.0), names=("P", "u") if first else ("K", "P", "x", "u"))
        cpu = {"value": len(idx) / dt, "unit": "instances/s", "cores": int(ref["threads"]), "kind": "oracle",
               "sample": "%d instances of the same workload, every (seq, head) covered" % len(idx),
               "seconds": dt, "parity_max_rel_err": errs, "speedup_gpu_over_cpu": value / (len(idx) / dt)}
        del ref

    line = {"metric": "lqr_instances_per_sec", "value": value, "unit": "instances/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "tf32" if kname == "riccati_umma" else "f32",
            "data": "synthetic",
            "config": {"workload": c["name"], "n": n, "m": m, "H": H, "instances": N, "batch": list(c["batch"]),
                       "q_x0_dtype": c["q_dtype"], "output_dtype": "bf16" if obf else "f32",
                       "q_operand": "U U'/8 + diag(d) factors" if lowrank else "dense", "time_varying": list(c.get("tv", ())), "outputs": list(want), "method": method_name, "kernel": kname,
                       "l2": "inputs+outputs per step exceed L2 (%.2f GB)" % (alg_bytes / 1e9)
                       if alg_bytes > 256e6 else "workload fits L2: a 192 MB buffer is written between timed steps"},
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "launches_per_step": launches_per_step, "clocks": clocks,
            "ms_per_step_percentiles": {"p20": float(np.percentile(per_step, 20)), "p50": float(np.percentile(per_step, 50)),
                                        "p80": float(np.percentile(per_step, 80))}}
    solver.close()
    del out, w
    torch.cuda.empty_cache()
    return line


# side measurements of the default run: (workload, method)
SIDE_RUNS = (("cfg0", "auto"), ("cfg1", "auto"), ("cfg2", "auto"), ("cfg3", "auto"), ("cfg3", "scan"))


def spawn_ranks(n):
    """`--gpus N` outside a launcher: start N ranks of this script, one per GPU, over NCCL on this node."""
    raise SystemExit(sharding.launch_ranks(n, __file__, sys.argv[1:]))


def run_layer_sweep(args):
    """--sweep with a layer workload: the horizon x batch grid of the paper's efficiency benchmark (d = 16,
    T in 2^4..2^11, B in 2^4..2^13) for the layer solve and for the sigma-product baseline, forward pass only.
    One JSON line with a row per grid point: median time of 5 solves, nominal B T d^3 throughput (the paper's
    convention), and the error of u_1 against the float64 oracle on up to 64 instances."""
    from paper_2603_09221_b200 import lqr
    from oracle import ttc_layer as lay
    key = args.workload
    c = workloads.LAYER_CONFIGS[key]
    n = c["n"]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    grid_T = [16, 64, 256, 1024, 2048] if not args.horizon else [args.horizon]
    grid_B = [16, 128, 1024, 8192]
    flush = torch.empty(192 * 1024 * 1024, dtype=torch.uint8, device=dev)
    rows = []
    for B in grid_B:
        batch = (1, 16, max(1, B // 16))
        w = workloads.make_layer_workload(key, device=dev, batch=batch)
        N = w["N"]
        ins = [w[k] for k in workloads.LAYER_KEYS]
        u1 = torch.empty((N, n), device=dev)
        P0 = torch.empty((N, n, n), device=dev)
        info = torch.empty((N,), dtype=torch.int32, device=dev)
        idx = np.unique(np.linspace(0, N - 1, min(N, 64)).astype(np.int64))
        f64 = lambda k, sel=None: (w[k] if sel is None else w[k][torch.as_tensor(sel, device=dev)]).to(torch.float64).cpu().numpy()
        for T in grid_T:
            solver = lqr.LqrSolver(n, n, T, batch, device=0)
            ref = lay.solve_batch(*(f64(k, idx) for k in workloads.LAYER_KEYS[:9]), f64("B_basis"), f64("Q_basis"), T)
            row = {"B": N, "T": T}
            for name, fn in (("recursion", solver.solve_layer), ("sigma_baseline", solver.solve_layer_sigma_baseline)):
                times = []
                for it in range(8):
                    flush.fill_(it)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn(*ins, T, u1=u1, P0=P0, info=info)
                    e1.record()
                    torch.cuda.synchronize(dev)
                    if it >= 3:
                        times.append(e0.elapsed_time(e1))
                ms = statistics.median(times)
                err = np.abs(u1.cpu()[torch.as_tensor(idx)].double().numpy() - ref["u1"]).max(axis=1) / np.abs(ref["u1"]).max(axis=1)
                row[name] = {"ms": ms, "nominal_BTd3_gflops": N * T * n ** 3 / (ms * 1e-3) / 1e9,
                             "u1_rel_err_median": float(np.nanmedian(err)), "u1_rel_err_max": float(np.nanmax(err))}
            rows.append(row)
            solver.close()
    print(json.dumps({"metric": "lqr_instances_per_sec", "sweep": key, "d": n, "data": "synthetic", "unit": "ms per solve",
                      "note": "forward pass only; B x T grid of the paper's efficiency benchmark; a 192 MB buffer is written "
                              "between timed solves", "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="", help="one workload only (cfg0..cfg4, tv16, tv32, layer16, layer32, grad16); "
                    "default: cfg4 as the headline plus short side measurements of cfg0..cfg3")
    ap.add_argument("--method", default="auto", choices=["auto", "riccati", "scan", "sigma"],
                    help="sigma: layer workloads only, the row-normalised reverse symplectic product (baseline)")
    ap.add_argument("--math", default="auto", choices=["auto", "fp32", "tf32"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-sample", type=int, default=4096, help="instances the oracle is timed on and parity is checked on")
    ap.add_argument("--ref-instances", type=int, default=2048)
    ap.add_argument("--tokens", type=int, default=0, help="override the token count (small profiling captures)")
    ap.add_argument("--horizon", type=int, default=0, help="layer workloads: override the planning horizon T (sweeps)")
    ap.add_argument("--batch", default="", help="layer and gradient workloads: override the batch as SxHxT, e.g. 1x16x64 (sweeps)")
    ap.add_argument("--per-token", action="store_true", help="grad16: A_t, B_t, R_t per token instead of per head")
    ap.add_argument("--out-dtype", default="f32", choices=["f32", "bf16"], help="bfloat16 K, P, x, u (TTC_OUT_BF16)")
    ap.add_argument("--lowrank-q", action="store_true", help="cfg4: hand Q over as its factors (ttc_lqr_solve_lowrank_q)")
    ap.add_argument("--grad", action="store_true", help="layer workloads: time ttc_lqr_layer_grad (every gradient requested)")
    ap.add_argument("--sweep", action="store_true", help="layer workloads: horizon x batch grid, recursion and sigma baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sides", action="store_true", help="default run: skip the side measurements of cfg0..cfg3")
    ap.add_argument("--no-peaks", action="store_true", help="skip the in-run FP32 / TF32 peak measurement (derived peaks are used)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        spawn_ranks(args.gpus)
    default_run = args.workload == ""
    if default_run:
        args.workload = "cfg4"
    if args.workload in workloads.LAYER_CONFIGS:
        if args.sweep:
            run_layer_sweep(args)
        else:
            run_layer(args)
        return
    if workloads.TV_CONFIGS.get(args.workload, {}).get("grad"):
        run_grad(args)
        return
    tv_key = args.workload if args.workload in workloads.TV_CONFIGS else None
    cid = None if tv_key else int(args.workload.replace("cfg", ""))
    if args.impl == "reference":
        run_reference(args, cid, tv_key)
        return
    args.warmup = max(args.warmup, 3)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the solver has no CPU path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = world > 1
    if dist:
        import torch.distributed as td
        td.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    ctx = dict(dist=dist, world=world, rank=rank, local=local, dev=dev, peaks=measured_peaks(), run_peaks=None)
    if rank == 0 and not args.no_peaks:
        ctx["run_peaks"] = measure_run_peaks(local, dev)
    line = run_solve(args, args.workload, args.method, ctx)
    if rank == 0:
        line["measured_in_run"] = ctx["run_peaks"]
        if default_run and not args.no_sides and world == 1:
            sides = {}
            for wl, meth in SIDE_RUNS:
                r = run_solve(args, wl, meth, ctx, light=True)
                key = wl + ("_scan" if meth == "scan" else "")
                sides[key] = {"workload": r["config"]["workload"], "method": meth, "kernel": r["config"]["kernel"],
                              "ms_per_step": r["ms_per_step"], "value": r["value"], "unit": r["unit"],
                              "roofline": {k: r["roofline"][k] for k in ("bound", "frac", "peak", "unit", "achieved", "hbm_frac")},
                              "parity_max_rel_err": r["cpu_baseline"]["parity_max_rel_err"] if r["cpu_baseline"] else None,
                              "cpu_oracle_instances_per_s": r["cpu_baseline"]["value"] if r["cpu_baseline"] else None,
                              "clocks": r["clocks"], "gpu_launches": r["gpu_launches"]}
            line["configs"] = sides
        print(json.dumps(line))
    if dist:
        td.destroy_process_group()


if __name__ == "__main__":
    main()
