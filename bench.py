#!/usr/bin/env python
"""Benchmark of the NLR K-means iteration on B200.

  python bench.py --gpus N --steps K --warmup W [--config 1..5] [--impl reference]

A step is one whole pass of the hot path on one synthetic workload: the factor is reset to the
seeded starting point and gem_nlr_run takes the workload's configured number of iterations.
`value` = NLR iterations per second with X-hat, U0 resident in HBM (whole job: summed over ranks).
`e2e` = the same metric through gem_nlr_run_host: host buffers in, setup + iterations + labels,
U and labels copied back, all inside the timed region.

Without --config the line describes the largest single-GPU workload (config 5) and carries, under
`per_config`, the same objects for configs 1-4 measured in the same run (each config's buffers are
released before the next).  With --config C only that workload runs.
With N > 1 every rank runs an independent replica of the workload (weak scaling, no collective).
"""
from __future__ import annotations

import argparse
import gc
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
HEADLINE_CONFIG = 5            # the largest shape that fits one GPU
# nominal dense TF32 : bf16 tensor throughput on this part (1.1 : 2.25 PFLOP/s)
TF32_OVER_BF16 = 1.1 / 2.25
# the CPU-baseline leg times the oracle on about this much FP64 work per iteration (rows are cut to fit)
CPU_SAMPLE_FLOPS = 1.2e11


def _measured():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except Exception:
        return None


def _peaks():
    """(HBM GB/s, bf16 sustained TFLOP/s, kind)."""
    m = _measured()
    if m:
        return float(m["hbm_gbs"]), float(m["bf16_tflops_sustained"]), "measured"
    return 6650.0, 1400.0, "fallback"


# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the ncu captures summarised under
# profiles/ (the file named in each entry says at which kernel source state and size it was taken;
# configs 3, 4, 5 are captured at reduced n and scaled by n: every row is read and written once per launch).
# Keyed by (n, d, r, kernel path) -> {phase: (bytes, profile file)}; anything else reports null.
NCU_TRAFFIC = {
    (1_000_000, 128, 16, "mma.tf32x3"): {
        "second": (635.9e6, "profiles/mma_tf32x3_128x16_config2_medium.md"),
        "first": (587.1e6, "profiles/mma_tf32x3_128x16_config2_medium.md")},
    (10_000_000, 64, 100, "f16x3"): {
        "second": (10.36e9, "profiles/tcgen05_64x100_config3_many_cluster.md"),
        "first": (7.29e9, "profiles/tcgen05_64x100_config3_many_cluster.md")},
    # first phase of the tiled family: the first-product kernel alone (the separate vector pass reads U once more)
    (2_000_000, 768, 1000, "f16x3.tiled"): {
        "second": (21.51e9, "profiles/f16x3_tiled_768x1000_config4_embedding.md"),
        "first": (16.59e9, "profiles/f16x3_tiled_768x1000_config4_embedding.md")},
    (100_000_000, 32, 8, "ffma"): {
        "second": (19.50e9, "profiles/ffma_32x8_config5_massive.md"),
        "first": (16.81e9, "profiles/ffma_32x8_config5_massive.md")},
}


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
            self._halt.wait(0.1)

    def finish(self) -> dict:
        self._halt.set()
        self.join(timeout=6)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        pw = [float(r[2]) for r in self.rows if len(r) >= 7 and r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 7 for i in range(4)
                          if r[3 + i].lower().startswith("active")})
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(pw)) if pw else None, "reasons": reasons, "samples": len(sm)}


def algorithmic_bytes(n, d, r):
    """B_alg per iteration: X-hat read by both products, U read by the first, read + written by the
    second, ytilde read twice and ybar written + read (written ytilde only when the gate fires)."""
    return 8 * n * d + 12 * n * r + 16 * n


def minimal_bytes(n, d, r):
    """B_min per iteration: two passes over X-hat plus one read and one write of U."""
    return 8 * n * d + 8 * n * r


def first_phase_bytes(n, d, r):
    """Vector work + first product: X-hat and U read, ytilde read, ybar written."""
    return 4 * n * d + 4 * n * r + 8 * n


def second_product_bytes(n, d, r):
    """The fused second-product kernel alone: X-hat and U read, U written, ybar read."""
    return 4 * n * d + 8 * n * r + 4 * n


def workload_name(spec, r, T=None):
    s = f"{spec.name}: n={spec.n} d={spec.d} K={spec.K} r={r}"
    return s if T is None else s + f", {T} iterations per step"


# ---------------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------------
def oracle_sample_rows(n, d, K):
    """Rows of the bounded sample the oracle is timed on: all n when one iteration is at most
    CPU_SAMPLE_FLOPS of FP64 work (4 n d K), else a leading slice of that much work."""
    m = int(CPU_SAMPLE_FLOPS / (4.0 * d * K))
    m = max(4096, m)
    return n if m >= n else m


def time_oracle(X, U0, K, hp, warm, iters, budget_s=None):
    """Iterations/s of the oracle on (X, U0) as given: `warm` untimed iterations, then up to `iters`
    timed ones (at least one; stops early when budget_s is spent).  Returns (it/s, timed count)."""
    import oracle
    Xhat, _, _ = oracle.normalize(X)
    st = oracle.State(Xhat, U0)
    for _ in range(warm):
        st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
    t0 = time.perf_counter()
    k = 0
    while k < iters and (k < 1 or budget_s is None or time.perf_counter() - t0 < budget_s):
        st.step(K, hp["alpha"], hp["beta"], hp["eps_d"], hp["eps_c"], 10 ** 9)
        k += 1
    dt = time.perf_counter() - t0
    return k / dt, k


def cpu_baseline_leg(spec, X_host, U0_host, hp, warm=1, iters=3, budget_s=8.0):
    """The oracle as it stands on the host cores, on a bounded sample of the same workload: the first m
    rows (m = n when an iteration is cheap enough), warmed up, timed the way the reference arm times it.
    Work per iteration is exactly linear in the rows, so a slice's rate times m / n is the full-size rate."""
    import oracle
    n, d, K = spec.n, spec.d, spec.K
    m = oracle_sample_rows(n, d, K)
    X = X_host[:m]
    U0 = U0_host[:m]
    if m < n:
        U0 = np.array(U0, copy=True)
        U0 *= np.float32(np.sqrt(K / np.sum(U0.astype(np.float64) ** 2)))     # keep the slice feasible
    rate, k = time_oracle(np.ascontiguousarray(X), np.ascontiguousarray(U0), K, hp, warm, iters, budget_s)
    out = {"value": rate * m / n, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
           "sample": f"{k} timed iterations after {warm} warm-up on the first {m} of n={n} rows"
                     + ("" if m == n else f", rate scaled by {m}/{n} (work is linear in the rows)"),
           "extrapolated": m < n}
    return out


def run_reference(args, spec, hp):
    """The oracle, as it stands, on the host cores: every step is one iteration on the bounded sample
    (the leading rows of the same workload that the product arm's CPU leg uses)."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n, d, K = spec.n, spec.d, spec.K
    m = oracle_sample_rows(n, d, K)
    X, _, _ = synth.make_mixture(spec, rows=m)      # block-wise streams: the leading rows need not the rest
    U0 = synth.make_u0(m, K, K)                     # the same leading rows, scaled to be feasible on their own
    rate, k = time_oracle(X, U0, K, hp, args.warmup, args.steps, None)
    val = rate * m / n
    sample = (f"{k} timed iterations after {args.warmup} warm-up on the first {m} of n={n} rows (1 iteration per step)"
              + ("" if m == n else f", rate scaled by {m}/{n} (work is linear in the rows)"))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / val,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": workload_name(spec, K), "config_index": args.config or HEADLINE_CONFIG},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample,
                         "extrapolated": m < n},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ---------------------------------------------------------------------------------------------------
# roofline objects
# ---------------------------------------------------------------------------------------------------
def roofline_objects(n, d, r, path, ms_first, ms_second, it_s):
    """The `roofline` object: the phase that took longer in this run (first phase = vector work + first
    product + reductions, or the fused second product), the other phase under `other`, and the whole
    iteration under `iteration`."""
    hbm, bf16_sus, kind = _peaks()
    f16_pipe = "f16x3" in path and "tf32" not in path
    if f16_pipe:
        tpeak, tkind = bf16_sus, f"{kind} bf16 sustained (f16 pipe)"
    else:
        tpeak, tkind = bf16_sus * TF32_OVER_BF16, f"{kind} bf16 sustained x nominal tf32:bf16 ratio"
    mma_mult = 3 if ("tf32" in path or "f16x3" in path) else 0
    first_tc = mma_mult if not path.startswith("generic+") and not path.startswith("ffma+") else 0
    traffic = NCU_TRAFFIC.get((n, d, r, path), {})

    def phase(name, label, bytes_, mult, secs):
        t_hbm = bytes_ / (hbm * 1e9)
        flops = mult * 2.0 * n * d * r
        t_tc = flops / (tpeak * 1e12) if mult else 0.0
        tr = traffic.get(name)
        o = {"kernel": label, "ms_per_launch": secs * 1e3, "algorithmic_bytes": bytes_,
             "achieved_gbs": bytes_ / secs / 1e9, "frac_of_hbm": bytes_ / secs / 1e9 / hbm,
             "traffic": tr[0] if tr else None, "traffic_source": tr[1] if tr else None}
        if t_tc > t_hbm:
            ach = flops / secs / 1e12
            o.update({"bound": "tensor", "achieved": ach, "peak": tpeak, "unit": "TFLOP/s", "frac": ach / tpeak,
                      "peak_kind": tkind, "flops_per_launch": flops,
                      "flops_note": "3 tensor-core products (two-term operand split) per FP32-accurate product, 2ndr each",
                      "useful_tflops": 2.0 * n * d * r / secs / 1e12})
        else:
            ach = bytes_ / secs / 1e9
            o.update({"bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": ach / hbm,
                      "peak_kind": kind + " copy bandwidth"})
        return o

    p1 = phase("first", "first phase: vector work + first product Theta = X-hat^T U + reductions",
               first_phase_bytes(n, d, r), first_tc, ms_first * 1e-3)
    p2 = phase("second", "second product X-hat Theta + fused epilogue", second_product_bytes(n, d, r), mma_mult,
               ms_second * 1e-3)
    dom, oth = (p1, p2) if ms_first >= ms_second else (p2, p1)
    b_alg, b_min = algorithmic_bytes(n, d, r), minimal_bytes(n, d, r)
    mma_flops = (first_tc + mma_mult) * 2.0 * n * d * r
    t_hbm_it = b_alg / (hbm * 1e9)
    t_tc_it = mma_flops / (tpeak * 1e12) if mma_flops else 0.0
    iteration = {"ms": it_s * 1e3, "ms_between_phases": it_s * 1e3 - ms_first - ms_second,
                 "bound": "tensor" if t_tc_it > t_hbm_it else "hbm",
                 "frac": max(t_hbm_it, t_tc_it) / it_s,
                 "algorithmic_bytes": b_alg, "minimal_bytes": b_min,
                 "achieved_gbs": b_alg / it_s / 1e9, "frac_of_hbm_B_alg": b_alg / it_s / 1e9 / hbm,
                 "frac_of_hbm_B_min": b_min / it_s / 1e9 / hbm,
                 "frac_of_hbm_nominal_8TBs_B_alg": b_alg / it_s / 8e12,
                 "mma_flops": mma_flops, "achieved_tflops": mma_flops / it_s / 1e12,
                 "frac_of_tensor_peak": mma_flops / it_s / 1e12 / tpeak if mma_flops else 0.0,
                 "useful_tflops": 4.0 * n * d * r / it_s / 1e12, "tensor_peak_tflops": tpeak,
                 "tensor_peak_kind": tkind, "hbm_peak_gbs": hbm}
    out = dict(dom)
    out["other"] = oth
    out["iteration"] = iteration
    return out


# ---------------------------------------------------------------------------------------------------
# one workload on this rank's GPU
# ---------------------------------------------------------------------------------------------------
def bench_config(cfg, args, dev, rank, world, local, with_cpu, with_e2e):
    import torch
    import paper_2609_36074_b200 as gem
    from paper_2609_36074_b200 import replicas
    from paper_2609_36074_b200.binding import make_params

    spec = synth.config(cfg)
    if args.n:
        spec = spec.with_n(args.n)
    hp = synth.default_hparams(spec.K)
    T = args.iters or spec.iters
    n, d, K = spec.n, spec.d, spec.K
    r = K
    # every rank holds its own replica, seeded by rank
    rspec = replicas.replica_spec(spec, rank)
    X_host = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
    synth.make_mixture(rspec, out=X_host.numpy())
    U0_host = torch.empty((n, r), dtype=torch.float32, pin_memory=True)
    synth.make_u0(n, r, K, seed=rspec.seed, out=U0_host.numpy())

    # x_inplace = 2: the data buffer may be given up after setup (the tensor-core shapes then keep the row-major fp16
    # image pair in it instead of X-hat plus a separate pair in the workspace)
    kw = dict(alpha=hp["alpha"], beta=hp["beta"], eps_d=hp["eps_d"], eps_c=hp["eps_c"], T=T, T_min=T,
              precision=args.precision, x_inplace=2)
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
    # Per-phase split: the same steps once more with CUDA events around the two phases of every iteration.  The events
    # are kept out of the timed region above because they cost the short iterations 3-7 % (config 2: 300 event
    # records per 23 ms step); the phase times below therefore add up to slightly more than the iteration time.
    solver.profile(True)
    for _ in range(max(1, min(args.steps, 2))):
        one_step()
    torch.cuda.synchronize()
    ms_p1, ms_p2, prof_iters = solver.profile_read()
    solver.profile(False)
    ms = replicas.max_over_ranks(ms, dev)
    value = replicas.whole_job_rate(world, args.steps, T, ms)

    # labels (S7) timed on their own
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    lab = torch.empty(n, dtype=torch.int32, device=dev)
    solver.labels(lab)                      # untimed first call (module load)
    e0.record()
    solver.labels(lab)
    e1.record()
    torch.cuda.synchronize()
    labels_ms = e0.elapsed_time(e1)
    del lab
    path = solver.path()
    P = make_params(n, d, K, r=r, **kw)
    ws_bytes = gem.workspace_bytes(P)
    paper_bytes = gem.paper_storage_bytes(P)
    solver.destroy()
    del solver, Xd, U0d, Ud
    torch.cuda.empty_cache()

    # ---- host-buffer leg: the whole job through gem_nlr_run_host_timed ---------------------------
    e2e = None
    if with_e2e:
        buf = torch.empty(gem.host_job_device_bytes(P), dtype=torch.uint8, device=dev)
        Uh = torch.empty((n, r), dtype=torch.float32, pin_memory=True)
        labh = torch.empty(n, dtype=torch.int32, pin_memory=True)        # allocated outside the timed region
        reps = max(1, min(args.steps, 3))
        tot, wall, phases = 0.0, 0.0, np.zeros(5)
        for i in range(reps + 1):                                        # the first job is an untimed warm-up
            Uh.copy_(U0_host)
            torch.cuda.synchronize()
            ph = []
            t0 = time.perf_counter()
            e0.record()
            rc, _, a2, info2, it2 = gem.run_host(X_host, Uh, K, buf, labels=labh, phase_ms=ph, **kw)
            e1.record()
            torch.cuda.synchronize()
            t1 = time.perf_counter()
            if rc < 0:
                raise SystemExit(f"gem_nlr_run_host failed: {rc}")
            if i > 0:
                tot += e0.elapsed_time(e1)
                wall += (t1 - t0) * 1e3
                phases += np.array(ph)
        e2e_ms = replicas.max_over_ranks(tot / reps, dev)
        phases /= reps
        e2e = {"value": replicas.whole_job_rate(world, 1, T, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": 4 * n * (d + r), "d2h_bytes_per_step": 4 * n * (r + 1), "ms_per_job": e2e_ms,
               "breakdown_ms": {"h2d_x_ms": phases[0], "setup_ms": phases[1], "iterations_ms": phases[2],
                                "labels_and_d2h_ms": phases[3], "device_total_ms": phases[4],
                                "host_overhead_ms": wall / reps - phases[4], "wall_ms": wall / reps,
                                "h2d_gbs": 4 * n * d / max(phases[0], 1e-6) / 1e6,
                                "note": "setup overlaps the copy of U0; iterations include any wait for that copy; "
                                        "host overhead = wall clock around the call minus the device span "
                                        "(stream, event and pinned-record creation and release)"},
               "includes": "H2D of X and U0, mean + spectral norm + normalization (+ operand images), T iterations, "
                           "labels, D2H of U and labels"}
        del buf, Uh, labh
        torch.cuda.empty_cache()

    # ---- roofline: the longer of the two phases, the other beside it, the whole iteration ---------
    roofline = None
    if prof_iters > 0:
        roofline = roofline_objects(n, d, r, path, ms_p1 / prof_iters, ms_p2 / prof_iters,
                                    ms * 1e-3 / (args.steps * T))

    # ---- CPU oracle leg (rank 0, N = 1 only) ------------------------------------------------------
    cpu = None
    if with_cpu and rank == 0 and world == 1:
        cpu = cpu_baseline_leg(spec, X_host.numpy(), U0_host.numpy(), hp)

    out = {
        "value": value, "ms_per_step": ms / args.steps,
        "config": {"workload": workload_name(spec, r, T),
                   "l2": "inputs larger than L2" if 4 * n * d > 126e6 else "inputs fit in L2 (latency-bound case)",
                   "kernel_path": path, "replicas": world, "alpha": hp["alpha"], "beta": hp["beta"],
                   "phase_timing": "roofline phases from a second pass of the same steps with CUDA events around "
                                   "each phase; value and roofline.iteration from the timed steps without them"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
        "cpu_baseline": cpu,
        "setup": {"spectral_norm_ms": setup_ms, "a": a, "labels_ms": labels_ms},
        "footprint_bytes": {"X": 4 * n * d, "U": 4 * n * r, "workspace": ws_bytes,
                            "total": 4 * n * d + 4 * n * r + ws_bytes, "paper_storage_equation": paper_bytes},
        "last_iteration": {k: info[k] for k in ("t", "delta_hat", "rho", "fhat")},
    }
    del X_host, U0_host
    gc.collect()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=0,
                    help="1..5: run only this benchmark shape (default: config 5 as the headline plus configs 1-4 "
                         "under per_config)")
    ap.add_argument("--n", type=int, default=0, help="override n (reduced-n twin; for profiling captures)")
    ap.add_argument("--iters", type=int, default=0, help="override the iterations per step")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-per-config", action="store_true", help="headline workload only")
    ap.add_argument("--precision", type=int, default=-1)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours" and not args.n:
        print("note: fewer than 3 warm-up steps; the timing rules ask for at least 3", file=sys.stderr)

    head_cfg = args.config or HEADLINE_CONFIG
    spec = synth.config(head_cfg)
    if args.n:
        spec = spec.with_n(args.n)
    if args.impl == "reference":
        run_reference(args, spec, synth.default_hparams(spec.K))
        return

    import torch
    import torch.distributed as dist
    from paper_2609_36074_b200 import replicas
    rank, world, local = replicas.rank_world_local()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    head = bench_config(head_cfg, args, dev, rank, world, local, not args.no_cpu, not args.no_e2e)
    per_config = None
    if not args.config and not args.no_per_config and not args.n:
        per_config = []
        for c in (1, 2, 3, 4):
            o = bench_config(c, args, dev, rank, world, local, not args.no_cpu, not args.no_e2e)
            o["config_index"] = c
            per_config.append(o)

    if rank == 0:
        out = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        }
        for k in ("config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline", "setup", "footprint_bytes",
                  "last_iteration"):
            out[k] = head[k]
        out["config"]["config_index"] = head_cfg
        if per_config is not None:
            out["per_config"] = per_config
            out["roofline_frac_by_config"] = {str(head_cfg): head["roofline"]["iteration"]["frac"] if head["roofline"] else None,
                                              **{str(o["config_index"]): (o["roofline"]["iteration"]["frac"] if o["roofline"] else None)
                                                 for o in per_config}}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
