#!/usr/bin/env python
"""Benchmark of KurTail rotation learning on B200.

One "step" is one pass of the whole hot path -- loss, gradient and the step on
the orthogonal group -- over the resident calibration buffer, i.e. one
iteration of kt_fit.  The default workload is the Llama-2-7B-like attention
input (X bf16 65536 x 4096, Student-t(3) with 16 outlier channels x100, R
initialised to the normalised Hadamard matrix).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line.  The timed region is a fit of K steps, repeated back to back
until it has lasted --min-seconds (so that clocks settle and the clock record
holds many samples); ms_per_step is the mean over the repeats.  With --impl
reference the float64 CPU checker is timed on the host cores on a bounded sample
of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import re
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
NOMINAL_BF16_TFLOPS = 2250.0
KERNEL_SOURCES = {"gemm_tn_kernel": ("gemm_sm100.cuh", "sm100_prims.cuh"),
                  "fused_small_kernel": ("fused_small.cuh", "sm100_prims.cuh")}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(tflops_sustained=p.get("bf16_tflops_sustained"), tflops_burst=p.get("bf16_tflops"),
                    hbm_gbs=p.get("hbm_gbs"), source="measured")
    return dict(tflops_sustained=1400.0, tflops_burst=1590.0, hbm_gbs=6650.0, source="fallback")


def kernel_source_hash(kernel):
    """Fingerprint of the code a kernel is compiled from (comments and white space left out): DRAM counters taken
    from an older kernel are not quoted."""
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        with open(os.path.join(ROOT, "paper_2503_01483_b200", "csrc", name), "r") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update("".join(text.split()).encode())
    return h.hexdigest()[:16]


def recorded_traffic(kernel, role, d):
    """DRAM bytes (read + written) per token of one launch, from the ncu capture summarised under profiles/.

    profiles/dram_traffic.txt holds one line per captured launch:
        kernel role rows d bytes_read bytes_write fixed_bytes source_hash
    (fixed_bytes: the part that does not grow with the rows, e.g. the d x d operand).  Returns
    (bytes per row, fixed bytes) or None when there is no line for this kernel, role and width d, or when the
    kernel's source has changed since the counters were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    want = kernel_source_hash(kernel)
    with open(path) as f:
        for line in f:
            parts = line.split()
            if len(parts) != 8 or parts[0].startswith("#"):
                continue
            k, r, rows, dd, rd, wr, fixed, src = parts
            if k == kernel and r == role and int(dd) == int(d) and src == want:
                return (float(rd) + float(wr) - float(fixed)) / float(rows), float(fixed)
    return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=20):
        self.index = index
        self.period_ms = period_ms
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", str(self.period_ms)],
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
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], None, [], set()
        for t, line in self.rows:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                clk = float(parts[0]); mx = float(parts[1])
            except ValueError:
                continue
            if t0 <= t <= t1:
                sm.append(clk)
                try:
                    power.append(float(parts[2]))
                except ValueError:
                    pass
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        sm.sort()
        med = sm[len(sm) // 2] if sm else None
        return dict(sm_mhz=med, sm_max_mhz=mx, sm_mhz_min=sm[0] if sm else None, sm_mhz_p90=sm[int(len(sm) * 0.9)] if sm
                    else None, power_w_max=max(power) if power else None, samples=len(sm),
                    sample_period_ms=self.period_ms, reasons=sorted(reasons))


def threads_in_use():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_step_time(X64, R64, lr):
    """Seconds for the oracle's loss+gradient on the sample rows, and for its orthogonal step."""
    from oracle import kurtail_oracle as ko
    t0 = time.perf_counter()
    _, dR = ko.loss_grad(X64, R64)
    t_lg = time.perf_counter() - t0
    t0 = time.perf_counter()
    ko.orth_step(R64, dR, lr)
    t_orth = time.perf_counter() - t0
    return t_lg, t_orth


def cpu_baseline(sample_X, R_init, N_full, lr, d):
    """The oracle as it stands, on the host cores, on a bounded row sample (rows are independent, so the time of
    loss+gradient scales with N; the orthogonal step does not depend on N).  Timed on all cores numpy uses, and once
    more on one thread (loss+gradient on a quarter of the sample; the d^3 step only when it stays within seconds)."""
    import numpy as np
    X64 = sample_X.astype(np.float64)
    R64 = R_init.astype(np.float64)
    n_s = X64.shape[0]
    t_lg, t_orth = oracle_step_time(X64, R64, lr)
    t_full = t_lg * (N_full / n_s) + t_orth
    out = dict(value=N_full / t_full, unit="tokens/s", cores=threads_in_use(), kind="oracle",
               sample="float64 loss+gradient on %d of %d rows at full d (%.2f s) scaled to N, plus one full "
                      "orthogonal step (%.2f s)" % (n_s, N_full, t_lg, t_orth))
    try:
        from threadpoolctl import threadpool_limits
        from oracle import kurtail_oracle as ko
        n1 = max(16, n_s // 4)
        with threadpool_limits(limits=1):
            t0 = time.perf_counter()
            _, dR = ko.loss_grad(X64[:n1], R64)
            t1 = time.perf_counter() - t0
            # 14 d^3 float64 flops for the step's matrix products at ~10 GFLOP/s on one core
            if 14.0 * d ** 3 / 1e10 < 15.0:
                t0 = time.perf_counter()
                ko.orth_step(R64, dR, lr)
                t1o = time.perf_counter() - t0
                note = "one full orthogonal step (%.2f s)" % t1o
            else:
                t1o = t_orth * out["cores"]
                note = "the orthogonal step's all-core time x cores (%.1f s; too long to run on one thread here)" % t1o
        out["single_thread"] = dict(value=N_full / (t1 * (N_full / n1) + t1o), unit="tokens/s", cores=1,
                                    sample="loss+gradient on %d rows (%.2f s) scaled to N, plus %s" % (n1, t1, note))
    except Exception as e:  # threadpoolctl missing: the all-core figure stands alone
        out["single_thread"] = dict(value=None, note="not measured: %s" % type(e).__name__)
    return out


def run_reference(args, wl_name, d, N_full):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    import numpy as np
    from paper_2503_01483_b200 import synth
    from oracle import kurtail_oracle as ko
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_s = min(N_full, max(64, int(2.0e10 / (4.0 * d * d))))   # ~2e10 f64 flops of GEMM per step
    cfg = synth.config(WORKLOADS[wl_name][0], device="cpu", rows=n_s if wl_name != "kv_heads" else n_s // 32 * 32,
                       **({"layers": 1} if WORKLOADS[wl_name][0] in ("llama3_70b_sweep", "llama2_7b_r1_shared")
                          else {}))
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


def executed_flops_per_step(N, d, rep, fwd_terms, recompute, steps, fused):
    """Tensor-core flops one step really issues: the token GEMMs with every bf16 term of R and the recomputation,
    and the d x d products the device did not gate off (from the last step's choices and the fit's guard count)."""
    nd2 = 2.0 * N * d * d
    tok = nd2 * fwd_terms + nd2 + (nd2 * fwd_terms if recompute else 0.0)
    if fused:
        return tok, None
    d3 = 2.0 * float(d) ** 3
    st = rep.get("series_terms_last") or 0
    p0 = rep.get("p0_terms_last") or 0
    guards = rep.get("guards_run") or 0
    square = None
    if st:
        # A = dR R^T (1 term), P0 = W R (p0 terms), the further series terms, and per measuring step the 3-term
        # R^T R on the upper tiles (a little over half of the output) -- the polish product only runs when needed
        square = d3 * (1 + p0 + (st - 1)) + d3 * 3 * 0.53 * guards / max(steps, 1)
    return tok, square


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
                         "of one X sharded over the GPUs (kt_fit_sharded: an all-reduce of dR and of the loss per "
                         "step, enqueued by the library through its reduce hook; strong scaling)")
    ap.add_argument("--backward", default="stored", choices=["stored", "stored_f32", "recompute"],
                    help="kt_config.backward_mode: read back the Y the forward pass kept as float16 (default) or as "
                         "float32, or recompute Y in a second GEMM pass, so that Y never reaches memory")
    ap.add_argument("--loss-mode", default="token", choices=["token", "layer"],
                    help="kt_config.loss_mode: one kurtosis per token (headline) or one over the whole layer")
    ap.add_argument("--rmsnorm", action="store_true", help="kt_config.rmsnorm: RMSNorm after the rotation")
    ap.add_argument("--lr", type=float, default=0.0, help="override the workload's learning rate")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="repeat the timed K-step fit until the timed region has lasted this long (0: once)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the short side measurements (other modes and workloads) added to the line")
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
    kw = dict(device=dev, rows=N_full)
    if wl_cfg == "llama3_70b_sweep":
        kw["layers"] = args.layers if sweep else 1
    shared = args.workload == "llama2_7b_r1_shared"
    if shared:
        args.optimizer, args.loss_mode, args.rmsnorm = "adam", "layer", True
        kw["rows"] = None
    cfg = synth.config(wl_cfg, **kw)
    Xs = cfg["X"] if isinstance(cfg["X"], list) else [cfg["X"]]   # all layer buffers stay resident in HBM
    X = Xs[0]
    row_sharded = world > 1 and args.shard == "rows" and not sweep
    N_all = X.shape[0]
    if shared and world > 1:
        # every rank holds its own block of the stored buffers and gathers its share of every minibatch
        Xs = Xs[rank::world]
        X = Xs[0]
    elif row_sharded:
        # every rank generated the same X: keep this rank's block of rows (multiples of 128 except the last)
        per = (N_all // world + 127) // 128 * 128
        X = X[rank * per:min((rank + 1) * per, N_all)].contiguous()
    elif world > 1:
        # different data per rank: re-draw with a rank-dependent seed by rolling rows
        X = torch.roll(X, shifts=rank * 977, dims=0).contiguous()
    batch_local = SHARED_BATCH // world if (shared and row_sharded) else SHARED_BATCH
    N = SHARED_RPS * batch_local if shared else X.shape[0]
    lr = args.lr if args.lr > 0 else cfg["lr"]
    ctx_kw = dict(forward_terms=args.forward_terms, optimizer=1 if args.optimizer == "adam" else 0,
                  loss_mode=1 if args.loss_mode == "layer" else 0, rmsnorm=1 if args.rmsnorm else 0,
                  backward_mode={"stored": 0, "recompute": 1, "stored_f32": 2}[args.backward])
    ctx = kurtail.Context(dev, **ctx_kw)
    # (automatic: two bf16 terms of R for d <= 512, except that the single-pass d = 128 kernel takes one float16 term)
    fwd_terms = args.forward_terms if args.forward_terms in (1, 2) else (2 if 128 < d <= 512 else 1)

    def fresh_R(c=ctx, dd=d, init=cfg["init"]):
        if init == "hadamard":
            return c.init_rotation(dd, "hadamard")
        if init == "random_orthogonal":
            return synth.random_orthogonal(dd, seed=3, device=dev).contiguous()
        return c.init_rotation(dd, "identity")

    R = fresh_R()
    R0_host = R.cpu().numpy()
    hook = dist_util.all_reduce_hook(dist, dev) if row_sharded else None
    order = None
    if shared:
        # the shuffle: epochs of a seeded permutation of this rank's stored samples, cut into minibatches
        n_samples = len(Xs) * (Xs[0].shape[0] // SHARED_RPS)
        rng = np.random.default_rng(1234 + rank)

        def draw(steps):
            need = steps * batch_local
            return np.concatenate([rng.permutation(n_samples) for _ in range(need // n_samples + 1)])[:need].tolist()

    def one_fit(steps):
        """A fit of `steps` steps on this rank's data, continuing from the current R; returns the report."""
        if sweep:
            return ctx.fit_layers(Xs, sweep_Rs, steps, lr)[-1]
        if shared and row_sharded:
            return ctx.fit_shared_sharded(Xs, SHARED_RPS, draw(steps), batch_local, R, SHARED_RPS * SHARED_BATCH, hook,
                                          steps, lr)
        if shared:
            return ctx.fit_shared(Xs, SHARED_RPS, draw(steps), batch_local, R, steps, lr)
        if row_sharded:
            return ctx.fit_sharded(X, R, N_all, hook, steps, lr)
        return ctx.fit(X, R, steps, lr)

    sweep_Rs = [R]
    if sweep:
        ctx.fit(X, fresh_R(), max(args.warmup, 1), lr)   # warm-up steps on the first layer (also sizes the workspace)
        sweep_Rs = [R] + [fresh_R() for _ in Xs[1:]]
    else:
        one_fit(max(args.warmup, 1))      # warm-up steps (also sizes the workspace)
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    dist_util.barrier(dist)
    torch.cuda.synchronize()
    ctx.profile_begin()
    t_wall0 = time.time()
    times_ms, reps = [], []
    # every rank runs the same number of repeats: rank 0's clock decides, the others follow its count
    while True:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        rep = one_fit(args.steps)
        ev1.record()
        torch.cuda.synchronize()
        ms_r = dist_util.max_over_ranks(dist, ev0.elapsed_time(ev1), dev)
        times_ms.append(ms_r)
        reps.append(rep)
        go_on = 1.0 if (sum(times_ms) < args.min_seconds * 1e3 and len(times_ms) < 1000 and not sweep) else 0.0
        if dist is not None:
            t = torch.tensor([go_on], device=dev)
            dist.broadcast(t, src=0)
            go_on = float(t.item())
        if go_on == 0.0:
            break
    t_wall1 = time.time()
    prof = ctx.profile_end()
    dist_util.barrier(dist)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    n_layers = len(Xs) if sweep else 1
    repeats = len(times_ms)
    ms = sum(times_ms) / repeats                     # mean device time of one K-step fit (max over ranks each)
    ms_per_step = ms / (args.steps * n_layers)
    tokens_per_step = N_all if (row_sharded and not shared) else (SHARED_RPS * SHARED_BATCH if (shared and row_sharded)
                                                                   else world * N)
    value = tokens_per_step * args.steps * n_layers / (ms * 1e-3)
    rep = reps[-1]

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
    # (it holds 8192 launches; long runs overrun it, and then the split describes the steps it holds)
    steps_seen = max(g["fused"]["launches"] or g["forward"]["launches"], 1)
    share = {k: g[k]["ms"] / steps_seen / ms_per_step for k in g}
    timed_s = sum(times_ms) * 1e-3
    capped = bool(clocks and "sw_power_cap" in (clocks.get("reasons") or []))
    fused = g["fused"]["launches"] > 0
    if fused:
        # d = 128: the single-pass kernel reads X once; HBM bound.  Algorithmic bytes per launch = N * d * 2.
        t_f = g["fused"]["ms"] / g["fused"]["launches"] * 1e-3
        alg_bytes = 2.0 * N * d
        achieved = alg_bytes / t_f / 1e9
        peak = peaks["hbm_gbs"]
        tr = recorded_traffic("fused_small_kernel", "terms%d" % fwd_terms, d)
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": (tr[0] * N + tr[1]) if tr else None, "algorithmic_bytes": alg_bytes,
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
        # which measured cuBLAS figure the run compares with: the burst one for a short region that never met the
        # power cap, the sustained one for a region of a second or more or one whose clock record shows the cap
        use_burst = (not capped) and timed_s < 1.0
        peak = peaks["tflops_burst"] if use_burst else peaks["tflops_sustained"]
        trs = [recorded_traffic("gemm_tn_kernel", r, d) for r in
               ({"stored": "forward_stored", "stored_f32": "forward_stored_f32", "recompute": "forward"}[args.backward],
                "backward_b")]
        traffic = None
        if all(trs):
            traffic = sum(t[0] * N + t[1] for t in trs) / 2.0        # mean of the two token GEMMs, per launch
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                    "frac": (achieved / peak) if achieved else None, "traffic": traffic,
                    "algorithmic_bytes": 2.0 * N * d,
                    "frac_of_sustained_peak": (achieved / peaks["tflops_sustained"]) if achieved else None,
                    "frac_of_burst_peak": (achieved / peaks["tflops_burst"]) if achieved else None,
                    "frac_of_nominal_peak": (achieved / NOMINAL_BF16_TFLOPS) if achieved else None,
                    "kernel": "gemm_tn_kernel (forward + moments, backward-B; backward-A too when it recomputes Y): "
                              "2*N*d^2 flops per launch",
                    "peak_source": "%s cuBLAS bf16 GEMM, %s" % (
                        peaks["source"], "burst (timed region %.2f s, no power-cap sample)" % timed_s if use_burst else
                        "sustained (timed region %.2f s%s)" % (timed_s, ", sw_power_cap seen" if capped else "")),
                    "per_role_ms_per_launch": per_role, "share_of_step": share}

    tok_exec, sq_exec = executed_flops_per_step(N, d, rep, fwd_terms, args.backward == "recompute", args.steps, fused)
    s_iters = 2
    alg_flops = 4.0 * N * d * d + 2.0 * float(d) ** 3 * (2 + s_iters)
    out = {
        "metric": METRIC + " at d=%d" % d, "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "steps_per_s": 1e3 / ms_per_step,
        "repeats": repeats, "timed_region_s": timed_s,
        "ms_per_step_min": min(times_ms) / (args.steps * n_layers),
        "ms_per_step_max": max(times_ms) / (args.steps * n_layers),
        "higher_is_better": True, "scaling": "strong" if row_sharded else "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": args.workload, "N": N, "d": d, "R_init": cfg["init"], "lr": lr,
                   "optimizer": "cayley_" + args.optimizer, "loss_mode": args.loss_mode, "rmsnorm": bool(args.rmsnorm),
                   "backward": args.backward + {"stored": " (Y kept as float16 between the forward and the backward pass)",
                                                "stored_f32": " (Y kept as float32 between the two passes)",
                                                "recompute": " (Y never written)"}[args.backward],
                   "l2": "inputs (%.0f MiB of X per step) exceed the 126 MB L2" % (N * d * 2 / 2**20)
                   if N * d * 2 > 126e6 else "inputs fit in L2; no flush (small case)",
                   "parallelism": ("rows of one batch over the GPUs, kt_fit_sharded: all-reduce of dR and loss per "
                                   "step" if row_sharded else "one independent layer per GPU") if world > 1
                   else "single GPU",
                   **({"layers": n_layers, "steps_per_layer": args.steps, "resident_gib": n_layers * N * d * 2 / 2**30,
                       "sweep_seconds": ms * 1e-3} if sweep else {})},
        # useful work: the two token GEMMs and the step's d x d products as the method states them (s = 2 iterations)
        "algorithmic_tflops": alg_flops * (1 if row_sharded else world) / (ms_per_step * 1e-3) / 1e12,
        # what the tensor cores really issued: every bf16 term, the recomputation, the products the device kept
        "executed_tflops": ((tok_exec + (sq_exec or 0.0)) * (1 if row_sharded else world) / (ms_per_step * 1e-3) / 1e12),
        "executed_flops_per_step": {"token_gemms": tok_exec, "square_products": sq_exec},
        "kcycles_per_step": (ms_per_step * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
        "loss_first": reps[0]["loss_first"], "loss_last": rep["loss_last"], "orth_err": rep["orth_err"],
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
                              "rows_per_sample": SHARED_RPS, "batch_samples": batch_local,
                              "resident_gib": len(Xs) * Xs[0].shape[0] * d * 2 / 2**30})
    if not args.no_cpu_baseline and world == 1 and not shared:
        n_s = min(N, max(64, int(2.0e10 / (4.0 * d * d))))
        sample = X[:n_s].float().cpu().numpy()
        out["cpu_baseline"] = cpu_baseline(sample, R0_host, N, lr, d)

    # ---- short side measurements, so that one line carries the other modes and workloads too
    if world == 1 and not args.no_extras and args.workload == "llama2_7b_attn" and not args.rows:
        extras = {}

        def short_fit(c, Xw, Rw, steps, lr_w, warm=3, tries=3):
            """The fastest of `tries` fits of `steps` steps (these side figures follow minutes of power-capped work,
            and the part's clock right after it varies from one short run to the next)."""
            c.fit(Xw, Rw, warm, lr_w)
            best = None
            for _ in range(tries):
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c.profile_begin()
                a.record()
                r = c.fit(Xw, Rw, steps, lr_w)
                b.record()
                torch.cuda.synchronize()
                pr = c.profile_end()
                ms_t = a.elapsed_time(b) / steps
                if best is None or ms_t < best[0]:
                    best = (ms_t, r, pr)
            return best

        # (the first entry is the timed configuration itself, run the short way, so that the others have something of
        # their own kind to be compared with: the headline comes from seconds of power-capped work)
        for name, kwx in (("default_short_run", dict()),
                          ("backward_recompute", dict(backward_mode=1)), ("backward_stored_f32", dict(backward_mode=2)),
                          ("optimizer_adam", dict(optimizer=1)),
                          ("lr_10_full_series", dict())):
            c2 = kurtail.Context(dev, **kwx)
            ms_x, r_x, _ = short_fit(c2, X, fresh_R(c2), 20, 10.0 if name == "lr_10_full_series" else lr)
            extras[name] = {"ms_per_step": ms_x, "tokens_per_s": N / (ms_x * 1e-3), "steps": 20, "best_of": 3,
                            "series_terms_last": r_x["series_terms_last"], "p0_terms_last": r_x["p0_terms_last"],
                            "guards_run": r_x["guards_run"], "orth_err": r_x["orth_err"]}
            c2.close()
        ctx.close()
        del X, Xs, R
        torch.cuda.empty_cache()
        for wl, steps_w in (("kv_heads", 50), ("llama3_70b_layer", 10), ("llama3_8b_down", 6)):
            wcfg_name, dw, Nw = WORKLOADS[wl]
            kww = dict(device=dev, rows=Nw)
            if wcfg_name == "llama3_70b_sweep":
                kww["layers"] = 1
            wc = synth.config(wcfg_name, **kww)
            Xw = wc["X"][0] if isinstance(wc["X"], list) else wc["X"]
            c2 = kurtail.Context(dev)
            # (the random orthogonal start of the widest workload is a float64 QR of minutes on the host: the side
            # measurement starts from a float32 QR made on the device)
            if wc["init"] == "random_orthogonal":
                gq = torch.Generator(device=dev).manual_seed(3)
                Rw = torch.linalg.qr(torch.randn((dw, dw), device=dev, generator=gq))[0].contiguous()
            else:
                Rw = fresh_R(c2, dw, wc["init"])
            ms_x, r_x, pr = short_fit(c2, Xw, Rw, steps_w, wc["lr"])
            gg = pr["gemm"]
            ex = {"ms_per_step": ms_x, "tokens_per_s": Nw / (ms_x * 1e-3), "steps": steps_w, "best_of": 3, "N": Nw, "d": dw,
                  "orth_err": r_x["orth_err"]}
            if gg["fused"]["launches"]:
                t_f = gg["fused"]["ms"] / gg["fused"]["launches"] * 1e-3
                ex["single_pass_kernel_us"] = t_f * 1e6
                ex["hbm_frac_of_measured"] = 2.0 * Nw * dw / t_f / 1e9 / peaks["hbm_gbs"]
                # (what the kernel saturates is not HBM: per 32 KB tile of X it moves 192 KB through the SM's
                # 128-byte-per-clock shared-memory port -- TMA write, two products with both operands there, the
                # stores of G -- 1603 wavefronts counted against the 1700-1750 cycles a tile takes)
                ex["limiter"] = "shared-memory data path of the SM (6 bytes per byte of HBM)"
            else:
                tk = [gg[k] for k in ("forward", "backward_b")]
                t_l = sum(x["ms"] for x in tk) / max(sum(x["launches"] for x in tk), 1) * 1e-3
                ex["token_gemm_tflops"] = 2.0 * Nw * dw * dw / t_l / 1e12
                ex["square_share_of_step"] = gg["square"]["ms"] / steps_w / ms_x
            extras[wl] = ex
            c2.close()
            del Xw, Rw, wc
            torch.cuda.empty_cache()
        out["extras"] = extras
    print(json.dumps(out))
    dist_util.finalize(dist)


if __name__ == "__main__":
    main()
