#!/usr/bin/env python
"""Benchmark of the NLR K-means iteration on B200.

  python bench.py --gpus N --steps K --warmup W [--config 1..5] [--impl reference]

A step is one whole pass of the hot path on one synthetic workload: the factor is reset to the
seeded starting point and gem_nlr_run takes the workload's configured number of iterations.
`value` = NLR iterations per second with X-hat, U0 resident in HBM (whole job: summed over ranks).
`e2e` = the same metric through gem_nlr_run_host: host buffers in, setup + iterations + labels,
U and labels copied back, all inside the timed region.
With N > 1 every rank runs an independent replica of the workload (weak scaling, no collective).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "nlr_iterations_per_second"
UNIT = "iterations/s"


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            m = json.load(f)
        return float(m["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the second-product kernel, from the ncu
# captures summarised under profiles/ (config 2 captured at full size; configs 3, 4, 5 captured at
# n = 2e6 / 131072 / 1.6e7 rows and scaled by n: every row is read and written once per launch).
# Keyed by (n, d, r, kernel path); anything else reports null.
NCU_TRAFFIC_BYTES = {
    (1_000_000, 128, 16, "mma.tf32x3"): 640.0e6,
    (10_000_000, 64, 100, "f16x3"): 10.36e9,
    (2_000_000, 768, 1000, "f16x3.tiled"): 21.52e9,
    (100_000_000, 32, 8, "ffma"): 19.49e9,
}

# nominal dense TF32 : bf16 tensor throughput on this part (1.1 : 2.25 PFLOP/s)
TF32_OVER_BF16 = 1.1 / 2.25


def _tensor_peak_tf32():
    """TF32 tensor peak in TFLOP/s: the measured cuBLAS bf16 figure sustained under the power cap (the
    kernels are timed inside a step of seconds) times the nominal TF32 : bf16 ratio."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            m = json.load(f)
        return float(m["bf16_tflops_sustained"]) * TF32_OVER_BF16, "measured bf16 sustained x nominal tf32:bf16 ratio"
    except Exception:
        return 1400.0 * TF32_OVER_BF16, "fallback bf16 sustained x nominal tf32:bf16 ratio"


class ClockSampler(threading.Thread):
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.rows, self._halt = index, [], threading.Event()

    def run(self):
        while not self._halt.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.rows.append([c.strip() for c in out.strip().split(",")])
            except Exception:
                pass
            self._halt.wait(0.2)

    def finish(self) -> dict:
        self._halt.set()
        self.join(timeout=6)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 7 for i in range(4)
                          if r[3 + i].lower().startswith("active")})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def algorithmic_bytes(n, d, r):
    """Per iteration: X-hat read by both products, U read by the first, read + written by the
    second, ytilde read twice and ybar written + read (written ytilde only when the gate fires)."""
    return 8 * n * d + 12 * n * r + 16 * n


def second_product_bytes(n, d, r):
    """The fused second-product kernel alone: X-hat and U read, U written, ybar read."""
    return 4 * n * d + 8 * n * r + 4 * n


def run_reference(args, spec, hp):
    """The oracle, as it stands, on the host cores.  One step = one iteration at full n."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    X, _, _ = synth.make_mixture(spec)
    Xhat, a, _ = oracle.normalize(X)
    del X
    st = oracle.State(Xhat, synth.make_u0(spec.n, spec.K, spec.K))
    for _ in range(args.warmup):
        st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        st.step(spec.K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
    dt = time.perf_counter() - t0
    val = args.steps / dt
    sample = f"{args.steps} consecutive iterations at full n={spec.n} (1 iteration per step)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": f"{spec.name}: n={spec.n} d={spec.d} K={spec.K} r={spec.K}"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="1..5: which benchmark shape (default: medium mixture)")
    ap.add_argument("--n", type=int, default=0, help="override n (reduced-n twin; for profiling captures)")
    ap.add_argument("--iters", type=int, default=0, help="override the iterations per step")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--precision", type=int, default=-1)
    args = ap.parse_args()

    spec = synth.config(args.config)
    if args.n:
        spec = spec.with_n(args.n)
    hp = synth.default_hparams(spec.K)
    T = args.iters or spec.iters
    if args.impl == "reference":
        run_reference(args, spec, hp)
        return

    import torch
    import torch.distributed as dist
    import paper_2609_36074_b200 as gem
    from paper_2609_36074_b200.binding import make_params

    from paper_2609_36074_b200 import replicas
    rank, world, local = replicas.rank_world_local()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    n, d, K = spec.n, spec.d, spec.K
    r = K
    # every rank holds its own replica, seeded by rank
    rspec = replicas.replica_spec(spec, rank)
    X_host = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
    synth.make_mixture(rspec, out=X_host.numpy())
    U0_host = torch.empty((n, r), dtype=torch.float32, pin_memory=True)
    synth.make_u0(n, r, K, seed=rspec.seed, out=U0_host.numpy())

    kw = dict(alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=T, T_min=T,
              precision=args.precision)
    Xd = X_host.to(dev, non_blocking=True)
    U0d = U0_host.to(dev, non_blocking=True)
    Ud = torch.empty_like(U0d)
    Ud.copy_(U0d)
    solver = gem.GemNlr(Xd, Ud, K, **kw)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    ev[0].record()
    a = solver.spectral_norm()
    ev[1].record()
    torch.cuda.synchronize()
    setup_ms = ev[0].elapsed_time(ev[1])

    def one_step():
        Ud.copy_(U0d)
        solver.set_state(None, 0)
        rc, info, iters = solver.run()
        if rc < 0 or iters != T:
            raise SystemExit(f"gem_nlr_run failed: rc={rc} iters={iters} {solver.last_error()}")
        return info

    for _ in range(args.warmup):
        one_step()
    solver.profile(True)
    launches0 = solver.launch_count()
    torch.cuda.synchronize()
    replicas.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    ev[2].record()
    for _ in range(args.steps):
        info = one_step()
    ev[3].record()
    torch.cuda.synchronize()
    replicas.barrier()
    clocks = sampler.finish()
    ms = ev[2].elapsed_time(ev[3])
    launches = solver.launch_count() - launches0
    ms_p1, ms_p2, prof_iters = solver.profile_read()
    solver.profile(False)
    ms = replicas.max_over_ranks(ms, dev)
    value = replicas.whole_job_rate(world, args.steps, T, ms)

    # labels (S7) timed on their own
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    lab = torch.empty(n, dtype=torch.int32, device=dev)
    solver.labels(lab)                      # untimed first call (allocation, module load)
    e0.record()
    solver.labels(lab)
    e1.record()
    torch.cuda.synchronize()
    labels_ms = e0.elapsed_time(e1)
    del lab
    path = solver.path()
    P = make_params(n, d, K, r=r, **kw)
    ws_bytes = gem.workspace_bytes(P)
    solver.destroy()

    # ---- host-buffer leg: the whole job through gem_nlr_run_host -------------------------------
    e2e = None
    if not args.no_e2e:
        buf = torch.empty(gem.host_job_device_bytes(P), dtype=torch.uint8, device=dev)
        Uh = torch.empty((n, r), dtype=torch.float32, pin_memory=True)
        reps = max(1, min(args.steps, 3))
        tot = 0.0
        for i in range(reps + 1):
            Uh.copy_(U0_host)
            torch.cuda.synchronize()
            e0.record()
            rc, lab, a2, info2, it2 = gem.run_host(X_host, Uh, K, buf, **kw)
            e1.record()
            torch.cuda.synchronize()
            if rc < 0:
                raise SystemExit(f"gem_nlr_run_host failed: {rc}")
            if i > 0:
                tot += e0.elapsed_time(e1)
        e2e_ms = tot / reps
        e2e_ms = replicas.max_over_ranks(e2e_ms, dev)
        e2e = {"value": replicas.whole_job_rate(world, 1, T, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": 4 * n * (d + r),
               "d2h_bytes_per_step": 4 * n * (r + 1), "ms_per_job": e2e_ms,
               "includes": "H2D of X and U0, mean + power iteration + normalization, T iterations, labels, D2H of U and labels"}
        del buf

    # ---- roofline of the dominant kernel (the fused second product) ------------------------------
    peak, peak_kind = _peaks()
    roofline = None
    if prof_iters > 0:
        p2_s = ms_p2 * 1e-3 / prof_iters
        it_s = ms * 1e-3 / (args.steps * T)
        # MMA flops actually issued on the tensor-core paths: three products per useful product; the fp16 split
        # runs on the f16 pipe (peak = the measured bf16 figure), the TF32 split on the TF32 pipe
        if "f16x3" in path and "tf32" not in path:
            tpeak, tpeak_kind = _tensor_peak_tf32()
            tpeak, tpeak_kind = tpeak / TF32_OVER_BF16, "measured bf16 sustained (f16 pipe)"
        else:
            tpeak, tpeak_kind = _tensor_peak_tf32()
        mma_mult = 3 if ("tf32" in path or "f16x3" in path) else 0
        t_hbm2 = second_product_bytes(n, d, r) / (peak * 1e9)
        t_tc2 = mma_mult * 2.0 * n * d * r / (tpeak * 1e12)
        iteration = {"algorithmic_bytes": algorithmic_bytes(n, d, r),
                     "achieved_gbs": algorithmic_bytes(n, d, r) / it_s / 1e9,
                     "frac_of_peak": algorithmic_bytes(n, d, r) / it_s / 1e9 / peak,
                     "mma_flops": mma_mult * 4.0 * n * d * r,
                     "achieved_tflops": mma_mult * 4.0 * n * d * r / it_s / 1e12,
                     "frac_of_tensor_peak": mma_mult * 4.0 * n * d * r / it_s / 1e12 / tpeak,
                     "tensor_peak_tflops": tpeak}
        if t_tc2 > t_hbm2:
            ach = mma_mult * 2.0 * n * d * r / p2_s / 1e12
            roofline = {"bound": "tensor", "kernel": "second product + fused epilogue", "achieved": ach, "peak": tpeak,
                        "unit": "TFLOP/s", "frac": ach / tpeak, "peak_kind": tpeak_kind,
                        "flops_per_launch": mma_mult * 2.0 * n * d * r,
                        "flops_note": "3 tensor-core products (two-term operand split) per FP32-accurate product, 2ndr each",
                        "traffic": NCU_TRAFFIC_BYTES.get((n, d, r, path)), "ms_per_launch": p2_s * 1e3,
                        "first_phase_ms_per_iteration": ms_p1 / prof_iters, "iteration": iteration}
        else:
            ach = second_product_bytes(n, d, r) / p2_s / 1e9
            roofline = {"bound": "hbm", "kernel": "second product + fused epilogue", "achieved": ach, "peak": peak,
                        "unit": "GB/s", "frac": ach / peak, "peak_kind": peak_kind + " copy bandwidth",
                        "traffic": NCU_TRAFFIC_BYTES.get((n, d, r, path)), "ms_per_launch": p2_s * 1e3,
                        "first_phase_ms_per_iteration": ms_p1 / prof_iters, "iteration": iteration}

    # ---- CPU oracle leg (rank 0, N = 1 only) ------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        Xhat_h, _, _ = oracle.normalize(X_host.numpy())
        st = oracle.State(Xhat_h, U0_host.numpy())
        t0 = time.perf_counter()
        k = 0
        while k < 8 and (k < 1 or time.perf_counter() - t0 < 12.0):
            st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
            k += 1
        dt = time.perf_counter() - t0
        cpu = {"value": k / dt, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
               "sample": f"first {k} iterations at full n={n}"}

    if rank == 0:
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"{spec.name}: n={n} d={d} K={K} r={r}, {T} iterations per step",
                       "l2": "inputs larger than L2" if 4 * n * d > 126e6 else "inputs fit in L2 (latency-bound case)",
                       "kernel_path": path, "replicas": world, "alpha": hp["alpha"], "beta": hp["beta"]},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu,
            "setup": {"spectral_norm_ms": setup_ms, "a": a, "labels_ms": labels_ms},
            "footprint_bytes": {"X": 4 * n * d, "U": 4 * n * r, "workspace": ws_bytes},
            "last_iteration": {k: info[k] for k in ("t", "delta_hat", "rho", "fhat")},
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
