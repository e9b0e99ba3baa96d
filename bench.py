#!/usr/bin/env python
"""Benchmark of KurTail rotation learning on B200.

One "step" is one pass of the whole hot path -- loss, gradient and the step on
the orthogonal group -- over the resident calibration buffer, i.e. one
iteration of kt_fit.  The default workload is the Llama-2-7B-like attention
input (X bf16 65536 x 4096, Student-t(3) with 16 outlier channels x100, R
initialised to the normalised Hadamard matrix).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  With --impl reference the float64 CPU checker is timed on
the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "calibration tokens/s per rotation step"
WORKLOADS = {
    # name: (config name in synth, d, full N)
    "llama2_7b_attn": ("llama2_7b_attn", 4096, 65536),
    "tiny": ("tiny", 256, 2048),
    "kv_heads": ("kv_heads", 128, 32 * 65536),
    "llama3_8b_down": ("llama3_8b_down", 14336, 32768),
    "llama3_70b_layer": ("llama3_70b_sweep", 8192, 32768),
    # the whole layer-wise sweep: --layers resident layer buffers (80 by default), --steps steps per layer
    "llama3_70b_sweep": ("llama3_70b_sweep", 8192, 32768),
    # the paper's procedure for the shared rotation R1: 64 stored buffers (32 layers x 2 blocks) of 8192 tokens, every
    # step a shuffled minibatch of 32 samples of 2048 tokens (N = 65536 tokens per step), Cayley Adam, whole-batch
    # kurtosis after RMSNorm
    "llama2_7b_r1_shared": ("llama2_7b_r1_shared", 4096, 65536),
}
SHARED_RPS, SHARED_BATCH = 2048, 32


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(tflops_sustained=p.get("bf16_tflops_sustained"), tflops_burst=p.get("bf16_tflops"),
                    hbm_gbs=p.get("hbm_gbs"), source="measured")
    return dict(tflops_sustained=1400.0, tflops_burst=1590.0, hbm_gbs=6650.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for t, line in self.rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                clk = float(parts[0]); mx = float(parts[1])
            except ValueError:
                continue
            if t0 <= t <= t1 + 0.1:
                sm.append(clk)
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        sm.sort()
        med = sm[len(sm) // 2] if sm else None
        return dict(sm_mhz=med, sm_max_mhz=mx, samples=len(sm), reasons=sorted(reasons))


def oracle_step_time(X64, R64, lr, repeats=1):
    """Seconds for the oracle's loss+gradient on the sample rows, and for its orthogonal step."""
    from oracle import kurtail_oracle as ko
    t0 = time.perf_counter()
    for _ in range(repeats):
        _, dR = ko.loss_grad(X64, R64)
    t_lg = (time.perf_counter() - t0) / repeats
    t0 = time.perf_counter()
    ko.orth_step(R64, dR, lr)
    t_orth = time.perf_counter() - t0
    return t_lg, t_orth


def threads_in_use():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def cpu_baseline(sample_X, R_init, N_full, lr):
    """The oracle as it stands, on the host cores, on a bounded row sample (rows are independent,
    so loss+gradient time scales with N; the orthogonal step does not depend on N)."""
    import numpy as np
    X64 = sample_X.astype(np.float64)
    R64 = R_init.astype(np.float64)
    n_s = X64.shape[0]
    t_lg, t_orth = oracle_step_time(X64, R64, lr)
    t_full = t_lg * (N_full / n_s) + t_orth
    return dict(value=N_full / t_full, unit="tokens/s", cores=threads_in_use(), kind="oracle",
                sample="float64 loss+gradient on %d of %d rows at full d (%.2f s) scaled to N, plus one full "
                       "orthogonal step (%.2f s)" % (n_s, N_full, t_lg, t_orth))


def run_reference(args, wl_name, d, N_full):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    import numpy as np
    import torch
    from paper_2503_01483_b200 import synth
    from oracle import kurtail_oracle as ko
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_s = min(N_full, max(64, int(2.0e10 / (4.0 * d * d))))   # ~2e10 f64 flops of GEMM per step
    cfg = synth.config(WORKLOADS[wl_name][0], device="cpu", rows=n_s if wl_name != "kv_heads" else n_s // 32 * 32,
                       **({"layers": 1} if wl_name == "llama3_70b_layer" else {}))
    X = cfg["X"][0] if isinstance(cfg["X"], list) else cfg["X"]
    X64 = X.float().numpy().astype(np.float64)
    n_s = X64.shape[0]
    R64 = ko.hadamard(d) if cfg["init"] == "hadamard" else np.eye(d)
    lr = cfg["lr"]
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        _, dR = ko.loss_grad(X64, R64)
        t1 = time.perf_counter()
        R64, _, _ = ko.orth_step(R64, dR, lr)
        t2 = time.perf_counter()
        if it >= args.warmup:
            times.append(((t1 - t0) * (N_full / n_s) + (t2 - t1)))
    t_step = sum(times) / len(times)
    val = N_full / t_step
    cores = threads_in_use()
    sample = ("each step: float64 loss+gradient on %d of %d rows at full d, time scaled to N, plus one full "
              "orthogonal step" % (n_s, N_full))
    print(json.dumps({
        "impl": "reference", "metric": METRIC + " at d=%d" % d, "value": val, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl_name, "N": N_full, "d": d},
        "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b_attn", choices=sorted(WORKLOADS))
    ap.add_argument("--rows", type=int, default=0, help="override N (profiling on a small case)")
    ap.add_argument("--layers", type=int, default=80, help="layers of the llama3_70b_sweep workload")
    ap.add_argument("--forward-terms", type=int, default=0, help="kt_config.forward_terms (0 = automatic)")
    ap.add_argument("--optimizer", default="sgd", choices=["sgd", "adam"],
                    help="kt_config.optimizer: Cayley SGD (the headline configuration) or Cayley Adam")
    ap.add_argument("--shard", default="layers", choices=["layers", "rows"],
                    help="with --gpus N > 1: one independent layer per GPU (weak scaling, no collective), or the rows "
                         "of one X sharded over the GPUs with an all-reduce of dR per step (strong scaling)")
    ap.add_argument("--backward", default="stored", choices=["stored", "recompute"],
                    help="kt_config.backward_mode: read back the float32 Y the forward pass kept (default) or "
                         "recompute Y in a second GEMM pass")
    ap.add_argument("--loss-mode", default="token", choices=["token", "layer"],
                    help="kt_config.loss_mode: one kurtosis per token (headline) or one over the whole layer")
    ap.add_argument("--rmsnorm", action="store_true", help="kt_config.rmsnorm: row-normalise X first")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    wl_cfg, d, N_full = WORKLOADS[args.workload]
    if args.rows:
        N_full = args.rows
    if args.impl == "reference":
        run_reference(args, args.workload, d, N_full)
        return

    import numpy as np
    import torch
    from paper_2503_01483_b200 import build, kurtail, synth

    from paper_2503_01483_b200 import dist_util
    rank, local_rank, world = dist_util.env_rank()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    dist = dist_util.init("nccl", dev)
    if rank == 0:
        build.build()
    dist_util.barrier(dist)

    # each rank fits its own layer buffer (layers are independent: no data-path collective)
    sweep = args.workload == "llama3_70b_sweep"
    kw = dict(device=dev, rows=N_full if wl_cfg != "kv_heads" else N_full)
    if wl_cfg == "llama3_70b_sweep":
        kw["layers"] = args.layers if sweep else 1
    shared = args.workload == "llama2_7b_r1_shared"
    if shared:
        args.optimizer, args.loss_mode, args.rmsnorm = "adam", "layer", True
        kw["rows"] = None
    cfg = synth.config(wl_cfg, **kw)
    Xs = cfg["X"] if isinstance(cfg["X"], list) else [cfg["X"]]   # all layer buffers stay resident in HBM
    X = Xs[0]
    row_sharded = world > 1 and args.shard == "rows" and not sweep and not shared
    N_all = X.shape[0]
    if row_sharded:
        # every rank generated the same X: keep this rank's block of rows (multiples of 128 except the last)
        per = (N_all // world + 127) // 128 * 128
        X = X[rank * per:min((rank + 1) * per, N_all)].contiguous()
    elif world > 1:
        # different data per rank: re-draw with a rank-dependent seed by rolling rows
        X = torch.roll(X, shifts=rank * 977, dims=0).contiguous()
    N = SHARED_RPS * SHARED_BATCH if shared else X.shape[0]
    lr = cfg["lr"]
    ctx = kurtail.Context(dev, forward_terms=args.forward_terms, optimizer=1 if args.optimizer == "adam" else 0,
                          loss_mode=1 if args.loss_mode == "layer" else 0, rmsnorm=1 if args.rmsnorm else 0,
                          backward_mode=1 if args.backward == "recompute" else 0)

    def fresh_R():
        if cfg["init"] == "hadamard":
            return ctx.init_rotation(d, "hadamard")
        if cfg["init"] == "random_orthogonal":
            return synth.random_orthogonal(d, seed=3, device=dev).contiguous()
        return ctx.init_rotation(d, "identity")

    R = fresh_R()
    R0_host = R.cpu().numpy()
    if shared:
        # the shuffle: epochs of a seeded permutation of all stored samples, cut into minibatches
        n_samples = len(Xs) * (Xs[0].shape[0] // SHARED_RPS)
        rng = np.random.default_rng(1234 + rank)
        need = (max(args.warmup, 1) + args.steps) * SHARED_BATCH
        order = np.concatenate([rng.permutation(n_samples) for _ in range(need // n_samples + 1)])[:need].tolist()
        w = max(args.warmup, 1)
        ctx.fit_shared(Xs, SHARED_RPS, order[:w * SHARED_BATCH], SHARED_BATCH, R, w, lr)
        order = order[w * SHARED_BATCH:]
    elif row_sharded:
        dist_util.fit_row_sharded(ctx, X, R, max(args.warmup, 1), lr, dist, N_all)
    else:
        ctx.fit(X, R, max(args.warmup, 1), lr)          # warm-up steps (also sizes the workspace)
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    dist_util.barrier(dist)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ctx.profile_begin()
    t_wall0 = time.time()
    ev0.record()
    if sweep:
        Rs = [R] + [fresh_R() for _ in Xs[1:]]
        torch.cuda.synchronize()
        ev0.record()
        reps = ctx.fit_layers(Xs, Rs, args.steps, lr)
        rep = reps[-1]
    elif shared:
        rep = ctx.fit_shared(Xs, SHARED_RPS, order, SHARED_BATCH, R, args.steps, lr)
    elif row_sharded:
        hist = dist_util.fit_row_sharded(ctx, X, R, args.steps, lr, dist, N_all)
        rep = dict(loss_first=hist[0], loss_last=hist[-1], orth_err=ctx.orth_error(R), alpha_last=None,
                   w_norm_last=None, w_op_last=None, series_terms_last=None, p0_terms_last=None, guards_run=None)
    else:
        rep = ctx.fit(X, R, args.steps, lr)
    ev1.record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    prof = ctx.profile_end()
    ms = ev0.elapsed_time(ev1)
    ms = dist_util.max_over_ranks(dist, ms, dev)
    dist_util.barrier(dist)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    n_layers = len(Xs) if sweep else 1
    ms_per_step = ms / (args.steps * n_layers)
    value = (N_all if row_sharded else world * N) * args.steps * n_layers / (ms * 1e-3)

    # ---- end to end through kt_fit_host: pinned host X and R in, R out, copies inside the timed region
    e2e = None
    if not args.no_e2e and not sweep and not shared and not row_sharded:
        Xh = X.cpu().pin_memory()
        Rh = torch.from_numpy(R0_host.copy()).pin_memory()
        stage = torch.empty_like(X)
        Rdev = torch.empty_like(R)
        ctx.fit_host(Xh, stage, Rh, Rdev, 1, lr)      # warm the copy path
        Rh.copy_(torch.from_numpy(R0_host))
        torch.cuda.synchronize()
        dist_util.barrier(dist)
        t0 = time.perf_counter()
        ctx.fit_host(Xh, stage, Rh, Rdev, args.steps, lr)
        torch.cuda.synchronize()
        t_e2e = time.perf_counter() - t0
        t_e2e = dist_util.max_over_ranks(dist, t_e2e, dev)
        h2d = Xh.numel() * Xh.element_size() + Rh.numel() * 4
        d2h = Rh.numel() * 4
        e2e = {"value": world * N * args.steps / t_e2e, "unit": "tokens/s",
               "h2d_bytes_per_step": h2d / args.steps, "d2h_bytes_per_step": d2h / args.steps,
               "note": "one kt_fit_host call of %d steps: X and R copied host->device once, R copied back once; "
                       "bytes are totals divided by steps" % args.steps}
        del Xh, stage

    if rank != 0:
        dist_util.finalize(dist)
        return

    # ---- roofline of the dominant kernel
    peaks = measured_peaks()
    g = prof["gemm"]
    per_role = {k: (g[k]["ms"] / g[k]["launches"] if g[k]["launches"] else None) for k in g}
    # every step launches exactly one forward (or one single-pass) kernel: the steps the event window covered
    # (it holds 8192 launches; the 80-layer sweep overruns it, and then the split describes the steps it holds)
    steps_seen = max(g["fused"]["launches"] or g["forward"]["launches"], 1)
    share = {k: g[k]["ms"] / steps_seen / ms_per_step for k in g}
    if g["fused"]["launches"] > 0:
        # d = 128: the single-pass kernel reads X once; HBM bound.  Algorithmic bytes per launch = N * d * 2.
        t_f = g["fused"]["ms"] / g["fused"]["launches"] * 1e-3
        alg_bytes = 2.0 * N * d
        achieved = alg_bytes / t_f / 1e9
        peak = peaks["hbm_gbs"]
        # DRAM bytes per launch: ncu capture at 1 048 576 rows (268.4 MB algorithmic; read + written 272.8 MB with
        # R as two bf16 terms, the default, and 272.0 MB with one), scaled by N
        traffic = alg_bytes * ((272.0 if args.forward_terms == 1 else 272.8) / 268.435)
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": traffic,
                    "kernel": "fused_small_kernel (loss + gradient in one pass over X): N*d*2 bytes per launch",
                    "peak_source": "%s copy bandwidth" % peaks["source"],
                    "per_role_ms_per_launch": per_role, "share_of_step": share}
    else:
        # the three N x d x d tensor-core GEMMs of a step (forward, backward-A, backward-B): 2*N*d^2 flops each
        tok = [g[k] for k in ("forward", "backward_a", "backward_b")]
        n_launch = sum(x["launches"] for x in tok)
        t_tok = sum(x["ms"] for x in tok)
        flops_per_launch = 2.0 * N * d * d
        achieved = flops_per_launch / (t_tok / max(n_launch, 1) * 1e-3) / 1e12 if t_tok > 0 else None
        peak = peaks["tflops_sustained"]
        traffic = None
        if args.workload == "llama2_7b_attn" and not tok[1]["launches"]:
            # mean DRAM bytes per launch of the two token GEMMs (forward with its float32 Y store, backward-B): ncu
            # capture at N = 16384 (same d); the part that grows with N (everything but the 33.5 MB of R^T read by
            # the forward pass) is scaled by N / 16384
            var_mb = (392.9 + 246.7 - 33.5) + (628.4 + 61.5)
            traffic = (var_mb * (N / 16384.0) + 33.5) / 2.0 * 1e6
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                    "frac_of_burst_peak": (achieved / peaks["tflops_burst"]) if achieved else None,
                    "frac_of_nominal_peak": (achieved / 2250.0) if achieved else None,
                    "kernel": "gemm_tn_kernel (forward + moments, backward-B; backward-A too when it recomputes Y): "
                              "2*N*d^2 flops per launch",
                    "peak_source": "%s bf16 GEMM, sustained (kernel timed inside a long step)" % peaks["source"],
                    "per_role_ms_per_launch": per_role, "share_of_step": share}

    out = {
        "metric": METRIC + " at d=%d" % d, "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "steps_per_s": 1e3 / ms_per_step,
        "higher_is_better": True, "scaling": "strong" if row_sharded else "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "N": N, "d": d, "R_init": cfg["init"], "lr": lr,
                   "optimizer": "cayley_" + args.optimizer, "loss_mode": args.loss_mode, "rmsnorm": bool(args.rmsnorm),
                   "backward": args.backward,
                   "l2": "inputs (%.0f MiB of X per step) exceed the 126 MB L2" % (N * d * 2 / 2**20)
                   if N * d * 2 > 126e6 else "inputs fit in L2; no flush (small case)",
                   "parallelism": ("rows of one X over the GPUs, all-reduce of dR per step" if row_sharded else
                                   "one independent layer per GPU") if world > 1 else "single GPU",
                   **({"layers": n_layers, "steps_per_layer": args.steps, "resident_gib": n_layers * N * d * 2 / 2**30,
                       "sweep_seconds": ms * 1e-3} if sweep else {})},
        "algorithmic_tflops": (4.0 * N * d * d) * world / (ms_per_step * 1e-3) / 1e12,
        "loss_first": rep["loss_first"], "loss_last": rep["loss_last"], "orth_err": rep["orth_err"],
        "alpha_last": rep["alpha_last"], "w_norm_last": rep["w_norm_last"],
        "step_choices": {k: rep[k] for k in ("w_op_last", "series_terms_last", "p0_terms_last", "guards_run")},
        "gpu_launches": prof["launches_total"], "clocks": clocks, "roofline": roofline, "e2e": e2e,
    }

    if world == 1 and not sweep:
        # the 4-bit fake-quantisation error of the fitted rotation (two GEMM passes; outside the timed region)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ctx.quant4_error(X, R)
        q0.record()
        mse = ctx.quant4_error(X, R)
        q1.record()
        torch.cuda.synchronize()
        out["quant4_error"] = {"mse": mse, "ms": q0.elapsed_time(q1)}
        # share of tokens whose largest magnitude the fitted rotation lowers: against the un-rotated token and
        # against the rotation the fit started from
        out["rowmax_success"] = {"vs_unrotated": ctx.rowmax_success(X, R),
                                 "vs_init": ctx.rowmax_success(X, R, fresh_R())}
    if shared:
        out["config"].update({"buffers": len(Xs), "rows_per_buffer": int(Xs[0].shape[0]),
                              "rows_per_sample": SHARED_RPS, "batch_samples": SHARED_BATCH,
                              "resident_gib": len(Xs) * Xs[0].shape[0] * d * 2 / 2**30})
    if not args.no_cpu_baseline and world == 1 and not shared:
        n_s = min(N, max(64, int(2.0e10 / (4.0 * d * d))))
        sample = X[:n_s].float().cpu().numpy()
        out["cpu_baseline"] = cpu_baseline(sample, R0_host, N, lr)
    print(json.dumps(out))
    dist_util.finalize(dist)


if __name__ == "__main__":
    main()
