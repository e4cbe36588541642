#!/usr/bin/env python
"""Benchmark of the fused FEM energy+residual path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--nu-mode kl|nodal]
    python bench.py --impl reference ...      # the fp64 CPU oracle on the host cores
    python bench.py --workload burgers ...    # second workload: the paper's finite-difference Burgers loss

One "step" is one pass of the whole hot path over one synthetic batch: a single
``dn_energy_grad`` call (KL tables -> fused energy+residual kernel -> energy
finaliser).  Prints ONE JSON line (rank 0).  With N > 1 ranks every rank
processes its own batch of the same shape (samples are independent: weak
scaling, no collective on the data path).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2007_12792_b200 import inputs, sharding  # noqa: E402

METRIC = "fused FEM energy+residual Gelements/s"
UNIT = "Gelements/s"
FALLBACK_HBM_GBS = 6650.0
FP32_PEAK_LANE_OPS = 148 * 128 * 1.965e9     # SMs x FP32 lanes x max SM clock: the FP32 issue roof (lane-ops/s)
# Counters of the dominant kernel from the ncu captures summarised under profiles/: DRAM bytes per
# launch (dram__bytes_read.sum + dram__bytes_write.sum) and executed FP32 lane-operations per element
# (FADD + FMUL + FFMA + 2 FFMA2).  Each entry names the kernel source it was taken from and the first 16
# hex digits of its sha256: once that file changes the entry no longer applies and null is reported.
NCU_CAPTURES = {
    "strip2d:cfg2_2d_2048^2_b16_m6:kl": {"traffic": 500101632, "fp32_ops_per_element": 57.7,
                                          "src": "dn_strip2d.cu", "sha": "5ba6034b044c172f"},
    "strip2d:cfg2_2d_2048^2_b16_m6:klnodal": {"traffic": 500000000, "fp32_ops_per_element": 44.0,
                                               "src": "dn_strip2d.cu", "sha": "5ba6034b044c172f"},
    "strip2d:cfg2_2d_2048^2_b16_m6:nodal": {"traffic": 790611967, "fp32_ops_per_element": 35.9,
                                             "src": "dn_strip2d.cu", "sha": "5ba6034b044c172f"},
    "strip3d:cfg4_3d_256^3_b4_m3:kl": {"traffic": 609947136, "fp32_ops_per_element": 133.8,
                                        "src": "dn_strip3d.cu", "sha": "f6a30d05f0f96c9e"},
    "strip3d:cfg4_3d_256^3_b4_m3:nodal": {"traffic": 837124096, "fp32_ops_per_element": 142.2,
                                           "src": "dn_strip3d.cu", "sha": "f6a30d05f0f96c9e"},
    "strip3d:cfg4_3d_256^3_b4_m3:klnodal": {"traffic": 557637888, "fp32_ops_per_element": 145.9,
                                             "src": "dn_strip3d.cu", "sha": "f6a30d05f0f96c9e"},
    "strip3d:cfg3_3d_64^3_b32_m2:kl": {"traffic": 49059584, "fp32_ops_per_element": 129.6,
                                        "src": "dn_strip3d.cu", "sha": "f6a30d05f0f96c9e"},
    "row2d:cfg1_2d_256^2_b64_m4:kl": {"traffic": 17594624, "fp32_ops_per_element": 51.0,
                                       "src": "dn_row2d.cu", "sha": "cc267857ef1ac237"},
    "march:burgers_1024x1024_b64": {"traffic": 499482880, "fp32_ops_per_element": 26.3,
                                    "src": "dn_burgers.cu", "sha": "baf4524ba7aede8d"},
}


def ncu_capture(key):
    import hashlib
    c = NCU_CAPTURES.get(key)
    if not c:
        return None
    try:
        with open(os.path.join(ROOT, "paper_2007_12792_b200", "csrc", c["src"]), "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest()[:16] != c["sha"]:
                return None
    except OSError:
        return None
    return c


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.1] or [r for _, r in self.rows]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample_run(cfg: int, mode: str, target_seconds: float = 12.0, want_results: bool = False):
    """Times the oracle (as it stands) on a bounded sample of the workload: whole samples of the batch."""
    import oracle
    wl = inputs.WORKLOADS[cfg]
    nu_mode = {"kl": oracle.NU_KL_GAUSS, "nodal": oracle.NU_NODAL, "klnodal": oracle.NU_KL_NODAL}[mode]

    def run(samples):
        inp = inputs.make_inputs(cfg, samples=samples)
        nu = None
        if nu_mode == oracle.NU_NODAL:
            nu = oracle.kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, inp.kl_w).astype(np.float32)
        p = oracle.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=nu_mode, nu=nu,
                           kl_modes=inp.kl_modes, kl_w=inp.kl_w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
        t = time.perf_counter()
        res = oracle.energy_grad(p, inp.u)
        return time.perf_counter() - t, res

    t1, res = run([0])
    n = int(max(1, min(wl.batch, round(target_seconds / max(t1, 1e-3)))))
    if n > 1:
        t, res = run(list(range(n)))
    else:
        t = t1
    base = {"value": wl.elements * n / t / 1e9, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{n} of {wl.batch} samples of {wl.name} ({wl.elements * n} elements, energy + full residual), "
                      f"{t:.2f} s wall"}
    if want_results:
        return base, t, n, res[0], res[3]
    return base, t, n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = inputs.WORKLOADS[args.config]
    times, base, n = [], None, 1
    for it in range(args.warmup + args.steps):
        # each step is a bounded sample sized so that the whole run stays within a few minutes
        base, t, n = oracle_sample_run(args.config, args.nu_mode,
                                       target_seconds=max(0.5, min(4.0, 150.0 / (args.steps + args.warmup))))
        if it >= args.warmup:
            times.append(t)
    ms = 1e3 * sum(times) / len(times)
    value = wl.elements * n / (ms * 1e-3) / 1e9
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "nu_mode": args.nu_mode},
            "detail": {"step": f"oracle pass over {n} sample(s)"},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


BURGERS = {"nx": 1024, "nt": 1024, "batch": 64}       # the paper's first high-resolution example: 1024 x 1024, minibatch 64
BURGERS_METRIC = "Burgers FD loss+gradient Gnodes/s"
BURGERS_UNIT = "Gnodes/s"
BURGERS_NAME = "burgers_1024x1024_b64"


def burgers_oracle_sample_run(target_seconds: float = 12.0):
    """Times the numpy oracle of the Burgers loss on whole samples of the workload."""
    from oracle import burgers as ob
    nodes = BURGERS["nx"] * BURGERS["nt"]

    def run(n):
        inp = inputs.burgers_inputs(BURGERS["nx"], BURGERS["nt"], BURGERS["batch"], samples=range(n))
        t = time.perf_counter()
        ob.loss_grad(inp.u, inp.c.astype(np.float64), T=float(np.float32(0.2)))
        return time.perf_counter() - t

    t1 = run(1)
    n = int(max(1, min(BURGERS["batch"], round(target_seconds / max(t1, 1e-3)))))
    t = run(n) if n > 1 else t1
    return {"value": nodes * n / t / 1e9, "unit": BURGERS_UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n} of {BURGERS['batch']} samples of {BURGERS_NAME} ({nodes * n} nodes, loss + full gradient, "
                      f"numpy fp64), {t:.2f} s wall"}, t, n


def run_reference_burgers(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    times, base, n = [], None, 1
    for it in range(args.warmup + args.steps):
        base, t, n = burgers_oracle_sample_run(target_seconds=max(0.5, min(4.0, 150.0 / (args.steps + args.warmup))))
        if it >= args.warmup:
            times.append(t)
    ms = 1e3 * sum(times) / len(times)
    value = BURGERS["nx"] * BURGERS["nt"] * n / (ms * 1e-3) / 1e9
    base["value"] = value
    print(json.dumps({"impl": "reference", "metric": BURGERS_METRIC, "value": value, "unit": BURGERS_UNIT,
                      "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                      "config": {"workload": BURGERS_NAME}, "detail": {"step": f"oracle pass over {n} sample(s)"},
                      "cpu_baseline": base,
                      "e2e": {"value": value, "unit": BURGERS_UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def main_burgers(args):
    """The paper's own loss (finite-difference Burgers residual) as a second workload: one step = one
    dn_burgers_loss_grad call (marching kernel + finaliser) over a minibatch of 64 fields of 1024 x 1024."""
    import torch
    import torch.distributed as dist
    from paper_2007_12792_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()
    nx, nt, bs = BURGERS["nx"], BURGERS["nt"], BURGERS["batch"]
    inp = inputs.burgers_inputs(nx, nt, world * bs, samples=sharding.minibatch_indices(world * bs, world * bs, world, rank, 0))
    u = torch.from_numpy(inp.u).cuda()
    c = torch.from_numpy(inp.c).cuda()
    g = torch.empty_like(u)
    L = torch.empty(bs, device="cuda")
    gL = torch.full((bs,), 1.0 / bs, device="cuda")            # gradient of the minibatch mean
    prob = B.Burgers(nx=nx, nt=nt, batch=bs, c=c, T=float(np.float32(0.2)), lam=1.0)
    ws = B.new_burgers_workspace(prob)
    cs = prob.c_struct()
    field_bytes = u.numel() * 4                                # 256 MiB in, 256 MiB out: larger than L2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K = args.steps
    ev_step = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    ev_main = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b_ in ev_step + ev_main:
        a.record(); b_.record()
    for _ in range(args.warmup):
        B.dn_burgers_loss_grad(prob, u, gL, L, None, g, ws, _cstruct=cs)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    t0 = time.time()
    for k in range(K):
        ev_step[k][0].record()
        B.dn_burgers_loss_grad(prob, u, gL, L, None, g, ws, event_before=ev_main[k][0], event_after=ev_main[k][1], _cstruct=cs)
        ev_step[k][1].record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    step_ms = sum(a.elapsed_time(b_) for a, b_ in ev_step) / K
    main_ms = sum(a.elapsed_time(b_) for a, b_ in ev_main) / K
    Lsum = float(L.double().sum())

    u_h = torch.from_numpy(inp.u).pin_memory()
    c_h = torch.from_numpy(inp.c).pin_memory()
    gL_h = gL.cpu().pin_memory()
    g_h = torch.empty(u.shape).pin_memory()
    L_h = torch.empty(bs).pin_memory()
    prob_h = B.Burgers(nx=nx, nt=nt, batch=bs, c=c_h, T=float(np.float32(0.2)), lam=1.0)
    staging = B.new_burgers_host_staging(prob_h)
    B.dn_burgers_loss_grad_host(prob_h, u_h, gL_h, L_h, None, g_h, staging)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        B.dn_burgers_loss_grad_host(prob_h, u_h, gL_h, L_h, None, g_h, staging)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
    step_ms, main_ms, e2e_ms = sharding.max_over_ranks([step_ms, main_ms, e2e_ms])
    Lmean = sharding.mean_over_ranks(Lsum, bs)
    if rank == 0:
        peak, peak_kind = measured_peak()
        nodes = nx * nt * bs
        alg_bytes = 8 * nodes
        achieved = alg_bytes / (main_ms * 1e-3) / 1e9
        cap = ncu_capture(f"march:{BURGERS_NAME}")
        line = {
            "metric": BURGERS_METRIC, "value": world * nodes / (step_ms * 1e-3) / 1e9, "unit": BURGERS_UNIT, "n_gpus": world,
            "steps": K, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": BURGERS_NAME},
            "detail": {"kernel_path": B.dn_burgers_path_name(prob, u, g), "nodes_per_step_per_gpu": nodes,
                       "sharding": "independent batches per rank", "l2": "inputs larger than L2"},
            "clocks": clocks,
            "e2e": {"value": world * nodes / (e2e_ms * 1e-3) / 1e9, "unit": BURGERS_UNIT,
                    "h2d_bytes_per_step": field_bytes + 8 * bs, "d2h_bytes_per_step": field_bytes + 4 * bs,
                    "ms_per_step": e2e_ms, "steps": args.e2e_steps, "entry": "dn_burgers_loss_grad_host (pinned host buffers)"},
            "gpu_launches": 2 * K,
            "roofline": {"bound": "hbm", "kernel": "burgers_march_kernel", "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                         "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": main_ms,
                         "traffic": cap["traffic"] if cap else None},
            "checksum_L": Lsum, "mean_L_all_ranks": Lmean,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = burgers_oracle_sample_run()[0]
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


CG_ITERS = 25
CG_BYTES_PER_NODE_ITER = 52        # operator 8 + update (p, q, u, r, 1/diag read; u, r written) 28 + direction 16


def main_cg(args):
    """The discrete FEM solution by matrix-free preconditioned CG on the fused kernel: one step = one dn_cg_solve
    call of CG_ITERS iterations (set-up included: boundary faces, initial residual, probed diagonal)."""
    import torch
    import torch.distributed as dist
    from paper_2007_12792_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = inputs.WORKLOADS[args.config]
    inp = inputs.make_inputs(args.config, samples=sharding.minibatch_indices(world * wl.batch, world * wl.batch, world, rank, 0))
    w = torch.from_numpy(inp.kl_w).cuda()
    u0 = torch.from_numpy(inp.u).cuda()
    u = torch.empty_like(u0)
    prob = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=B.DN_NU_KL_GAUSS,
                     kl_modes=inp.kl_modes, kl_w=w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    ws = B.new_cg_workspace(prob)
    relres = torch.empty(inp.batch, device="cuda")
    its = torch.empty(inp.batch, dtype=torch.int32, device="cuda")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(iters, reps):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for k in range(reps):
            u.copy_(u0)
            ev[k][0].record()
            B.dn_cg_solve(prob, u, iters, 0.0, relres, its, ws)
            ev[k][1].record()
        barrier()
        return sum(a.elapsed_time(b_) for a, b_ in ev) / reps

    timed(CG_ITERS, args.warmup)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    t0 = time.time()
    step_ms = timed(CG_ITERS, args.steps)
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    short_ms = timed(5, max(3, args.steps // 4))
    iter_ms = (step_ms - short_ms) / (CG_ITERS - 5)
    rel = float(relres.max())
    step_ms, iter_ms = sharding.max_over_ranks([step_ms, iter_ms])
    if rank == 0:
        peak, peak_kind = measured_peak()
        nodes = wl.nodes * inp.batch
        achieved = CG_BYTES_PER_NODE_ITER * nodes / (iter_ms * 1e-3) / 1e9
        launches_per_iter = (2 if B.dn_path_name(prob) in ("tiled3d", "strip3d") else 1) + 4    # fused kernel (3D: + seam fix-up) + 4 CG kernels
        print(json.dumps({
            "metric": "PCG Gnode-iterations/s", "value": world * nodes * CG_ITERS / (step_ms * 1e-3) / 1e9,
            "unit": "Gnode-iterations/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "nu_mode": "kl", "solver": f"dn_cg_solve, {CG_ITERS} iterations per step, set-up included",
                       "l2": "vectors larger than L2" if 4 * nodes > 2 * (126 << 20) else "vectors fit in L2"},
            "clocks": clocks, "ms_per_iteration": iter_ms, "relres_after_step": rel,
            "gpu_launches": args.steps * (CG_ITERS * launches_per_iter + 2 * (27 if inp.dim == 3 else 9) * 2 + 8),
            "roofline": {"bound": "hbm", "kernel": "one CG iteration (fused operator + cg_update_kernel + cg_direction_kernel)",
                         "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                         "frac": achieved / peak, "algorithmic_bytes_per_iteration": CG_BYTES_PER_NODE_ITER * nodes,
                         "traffic": None},
            "e2e": None, "cpu_baseline": None,
            "note": "e2e / cpu_baseline: the solve keeps every vector on the device; the oracle solves the assembled system directly"}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 0..4 (default: 2D 2048^2, batch 16)")
    ap.add_argument("--nu-mode", default="kl", choices=["kl", "nodal", "klnodal"],
                    help="kl: KL at Gauss points (default); nodal: stored nodal field; klnodal: KL at nodes inside the kernel")
    ap.add_argument("--workload", default="fem", choices=["fem", "burgers", "cg"],
                    help="fem: the Galerkin energy+residual path (default); burgers: the paper's finite-difference Burgers loss; "
                         "cg: matrix-free preconditioned CG on the fused kernel (workload --config, KL at Gauss points)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the device timing of the other target workloads and modes (default run only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference" and args.workload == "cg":
        if int(os.environ.get("RANK", "0")) == 0:
            print(json.dumps({"impl": "reference", "unavailable": "the oracle solves the assembled system directly; it has no CG iteration to time"}))
        return
    if args.impl == "reference":
        return run_reference_burgers(args) if args.workload == "burgers" else run_reference(args)
    if args.workload == "cg":
        return main_cg(args)
    if args.workload == "burgers":
        return main_burgers(args)

    import torch
    import torch.distributed as dist
    from paper_2007_12792_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()

    def device_run(cfg, nu_mode, K, warmup, sampler=None):
        """K timed steps of one workload on this rank's device: the step time (plain calls) and, from K more steps, the
        time of the fused kernel alone.  Returns the numbers and the tensors (for the parity check and the extras)."""
        wl = inputs.WORKLOADS[cfg]
        # every rank draws its own contiguous piece of the global mini-batch (world * B samples of the same recipe)
        inp = inputs.make_inputs(cfg, samples=sharding.minibatch_indices(world * wl.batch, world * wl.batch, world, rank, 0))
        u = torch.from_numpy(inp.u).cuda()
        w = torch.from_numpy(inp.kl_w).cuda()
        nu = None
        mode = {"kl": B.DN_NU_KL_GAUSS, "nodal": B.DN_NU_NODAL, "klnodal": B.DN_NU_KL_NODAL}[nu_mode]
        if mode == B.DN_NU_NODAL:
            nu = torch.empty_like(u)
            B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, w, nu)
        prob = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu,
                         kl_modes=inp.kl_modes, kl_w=w, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
        r = torch.empty_like(u)
        J = torch.empty(inp.batch, device="cuda")
        ws = B.new_workspace(prob)
        cs = prob.c_struct()
        field_bytes = u.numel() * 4
        l2_bytes = torch.cuda.get_device_properties(local).L2_cache_size
        traffic_bytes = 2 * field_bytes + (field_bytes if nu is not None else 0)
        flush = None
        if traffic_bytes < 2 * l2_bytes:
            flush = torch.empty(max(2 * l2_bytes, 256 << 20), dtype=torch.uint8, device="cuda")
        ev_step = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        ev_main = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for a, b_ in ev_step + ev_main:            # create the underlying CUDA events
            a.record(); b_.record()
        for _ in range(warmup):
            if flush is not None:
                flush.zero_()
            B.dn_energy_grad_traced(prob, u, None, J, r, ws, None, None, _cstruct=cs)
        barrier()
        if sampler is not None:
            sampler.start()
            time.sleep(0.15)
        t0 = time.time()
        # the K timed steps: the plain call a user makes (no events inside it).  Inputs larger than L2: one event pair
        # around all K steps; otherwise one pair per step, so that the L2 flush between steps stays outside the timing.
        if flush is None:
            ev_step[0][0].record()
            for k in range(K):
                B.dn_energy_grad_traced(prob, u, None, J, r, ws, None, None, _cstruct=cs)
            ev_step[0][1].record()
        else:
            for k in range(K):
                flush.zero_()
                ev_step[k][0].record()
                B.dn_energy_grad_traced(prob, u, None, J, r, ws, None, None, _cstruct=cs)
                ev_step[k][1].record()
        barrier()
        step_ms = (ev_step[0][0].elapsed_time(ev_step[0][1]) if flush is None
                   else sum(a.elapsed_time(b_) for a, b_ in ev_step)) / K
        # K more steps with events around the fused kernel alone (the roofline's kernel time)
        for k in range(K):
            if flush is not None:
                flush.zero_()
            B.dn_energy_grad_traced(prob, u, None, J, r, ws, ev_main[k][0], ev_main[k][1], _cstruct=cs)
        barrier()
        t1 = time.time()
        clocks = sampler.stop(t0, t1) if sampler is not None else None
        main_ms = sum(a.elapsed_time(b_) for a, b_ in ev_main) / K
        return {"wl": wl, "inp": inp, "u": u, "w": w, "nu": nu, "mode": mode, "prob": prob, "r": r, "J": J, "ws": ws, "cs": cs,
                "field_bytes": field_bytes, "flush": flush, "step_ms": step_ms, "main_ms": main_ms, "clocks": clocks,
                "nu_mode": nu_mode}

    def roofline_of(run, step_ms, main_ms):
        """The roofline objects of one device run (rank 0): HBM (the metric's roof) and FP32 issue."""
        wl, inp, mode = run["wl"], run["inp"], run["mode"]
        peak, peak_kind = measured_peak()
        elements = wl.elements * inp.batch
        nodes = wl.nodes * inp.batch
        alg_bytes = nodes * (12 if mode == B.DN_NU_NODAL else 8)
        achieved = alg_bytes / (main_ms * 1e-3) / 1e9
        path = B.dn_path_name(run["prob"])
        cap = ncu_capture(f"{path}:{wl.name}:{run['nu_mode']}")
        alu = None
        if cap:
            ops = cap["fp32_ops_per_element"] * elements / (main_ms * 1e-3)
            alu = {"bound": "alu", "achieved": ops / 1e12, "peak": FP32_PEAK_LANE_OPS / 1e12, "unit": "T FP32 lane-ops/s",
                   "frac": ops / FP32_PEAK_LANE_OPS, "fp32_ops_per_element": cap["fp32_ops_per_element"],
                   "note": "executed FP32 operations (ncu) / kernel time, against SMs x 128 lanes x max clock"}
        roof = {"bound": "hbm", "kernel": f"fused energy+residual ({path})", "achieved": achieved,
                "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms": main_ms,
                "traffic": cap["traffic"] if cap else None}
        return path, elements, roof, alu

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    K = args.steps
    sampler = ClockSampler(local) if rank == 0 else None
    run = device_run(args.config, args.nu_mode, K, args.warmup, sampler)
    wl, inp, u, w, nu, mode, prob, r, J, ws, cs = (run[k] for k in ("wl", "inp", "u", "w", "nu", "mode", "prob", "r", "J", "ws", "cs"))
    field_bytes, flush, step_ms, main_ms, clocks = (run[k] for k in ("field_bytes", "flush", "step_ms", "main_ms", "clocks"))
    Jsum = float(J.double().sum())

    # ---- the two small entry points of the path: diffusivity synthesis (4 B/node written) and the Dirichlet faces
    nu_tmp = nu if nu is not None else torch.empty_like(u)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    n_aux = 10
    B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, w, nu_tmp)
    ev[0].record()
    for _ in range(n_aux):
        B.dn_kl_field(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, inp.kl_modes, w, nu_tmp)
    ev[1].record()
    r_bc = r
    ev[2].record()
    for _ in range(n_aux):
        B.dn_apply_bc(inp.dim, inp.nx, inp.ny, inp.nz, inp.batch, 0.0, 0.0, 1, r_bc)      # r is zero there already
    ev[3].record()
    torch.cuda.synchronize()
    klf_ms = ev[0].elapsed_time(ev[1]) / n_aux
    bc_ms = ev[2].elapsed_time(ev[3]) / n_aux
    lines = inp.batch * inp.ny * inp.nz
    aux = {"dn_kl_field": {"us": 1e3 * klf_ms, "GB/s": field_bytes / (klf_ms * 1e-3) / 1e9, "bytes": field_bytes,
                           "note": "back-to-back calls; output larger than L2 only on the 256 MiB workloads"},
           "dn_apply_bc": {"us": 1e3 * bc_ms, "algorithmic_bytes": 2 * lines * 4, "sector_bytes": 2 * lines * 32}}
    if nu is None:
        del nu_tmp

    # ---- L2-resident workloads: also time warm (no flush) and as a replayed CUDA graph (launch-bound cases)
    extras = None
    if flush is not None:
        n_rep = 50
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(n_rep):
            B.dn_energy_grad_traced(prob, u, None, J, r, ws, None, None, _cstruct=cs)
        b_.record()
        torch.cuda.synchronize()
        warm_us = 1e3 * a.elapsed_time(b_) / n_rep
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                B.dn_energy_grad_traced(prob, u, None, J, r, ws, None, None, _cstruct=cs, stream=side)
        torch.cuda.current_stream().wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        a.record()
        for _ in range(n_rep):
            graph.replay()
        b_.record()
        torch.cuda.synchronize()
        extras = {"warm_us_per_call": warm_us, "graph_replay_us_per_call": 1e3 * a.elapsed_time(b_) / n_rep,
                  "note": "workload fits in L2: back-to-back calls without flush, and the same call replayed from a CUDA graph"}
    barrier()

    # ---- end to end: host buffers in, host buffers out, through the C-ABI host entry point ----------
    u_h = torch.from_numpy(inp.u).pin_memory()
    w_h = torch.from_numpy(inp.kl_w).pin_memory()
    nu_h = nu.cpu().pin_memory() if nu is not None else None
    r_h = torch.empty(u.shape).pin_memory()
    J_h = torch.empty(inp.batch).pin_memory()
    prob_h = B.Problem(dim=inp.dim, nx=inp.nx, ny=inp.ny, nz=inp.nz, batch=inp.batch, nu_mode=mode, nu=nu_h,
                       kl_modes=inp.kl_modes, kl_w=w_h, f_const=inp.f_const, bc_x0=inp.bc_x0, bc_x1=inp.bc_x1)
    staging = B.new_host_staging(prob_h)
    B.dn_energy_grad_host(prob_h, u_h, None, J_h, r_h, staging)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.e2e_steps):
        B.dn_energy_grad_host(prob_h, u_h, None, J_h, r_h, staging)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
    h2d = field_bytes + w.numel() * 4 + (field_bytes if nu is not None else 0)
    d2h = field_bytes + inp.batch * 4

    step_ms, main_ms, e2e_ms = sharding.max_over_ranks([step_ms, main_ms, e2e_ms])
    Jmean = sharding.mean_over_ranks(Jsum, inp.batch)          # the averaged loss of Algorithm 1 (one scalar all-reduce)

    # ---- the other target workloads and modes, device-timed in this process (single-GPU default run only)
    secondary = None
    if world == 1 and not args.no_secondary and args.config == 2 and args.nu_mode == "kl":
        secondary = []
        # ... and the three workloads that fit in L2, timed cold (L2 flushed between steps, outside the timed region)
        for cfg2, mode2 in ((4, "kl"), (4, "nodal"), (2, "nodal"), (2, "klnodal"), (0, "kl"), (1, "kl"), (3, "kl")):
            sub = device_run(cfg2, mode2, max(5, min(K, 20)), 3, ClockSampler(local))
            path2, elements2, roof2, alu2 = roofline_of(sub, sub["step_ms"], sub["main_ms"])
            secondary.append({"workload": sub["wl"].name, "nu_mode": mode2, "kernel_path": path2, "ms_per_step": sub["step_ms"],
                              "value": elements2 / (sub["step_ms"] * 1e-3) / 1e9, "unit": UNIT, "roofline": roof2,
                              "roofline_alu": alu2, "clocks": sub["clocks"], "checksum_J": float(sub["J"].double().sum()),
                              "l2": "inputs larger than L2" if sub["flush"] is None else "L2 flushed between steps"})
            del sub
            torch.cuda.empty_cache()

    if rank == 0:
        path, elements, roof, alu = roofline_of(run, step_ms, main_ms)
        line = {
            "metric": METRIC, "value": world * elements / (step_ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "nu_mode": args.nu_mode},        # the same keys in the reference arm's line
            "detail": {"kernel_path": path, "elements_per_step_per_gpu": elements, "sharding": "independent batches per rank",
                       "l2": "inputs larger than L2" if flush is None else "L2 flushed between steps"},
            "clocks": clocks,
            "e2e": {"value": world * elements / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": args.e2e_steps,
                    "entry": "dn_energy_grad_host (pinned host buffers)"},
            "gpu_launches": K * B.dn_launches_per_call(prob),
            "roofline": roof,
            "roofline_alu": alu,
            "checksum_J": Jsum, "mean_J_all_ranks": Jmean, "l2_resident_extras": extras, "aux_kernels": aux,
            "secondary": secondary,
        }
        if not args.no_cpu_baseline and world == 1:
            base, _, n, Jo, ro = oracle_sample_run(args.config, args.nu_mode, want_results=True)
            line["cpu_baseline"] = base
            # the device results of the timed run against the oracle's, on the samples the baseline just computed
            Jg = J[:n].cpu().numpy().astype(np.float64)
            rerr = 0.0
            for b_ in range(n):
                rerr = max(rerr, float(np.abs(r[b_].cpu().numpy() - ro[b_]).max()))
            line["parity"] = {"samples": n, "J_max_rel_err": float(np.max(np.abs(Jg - Jo) / np.abs(Jo))),
                              "r_max_err_over_max_abs_r": rerr / float(np.abs(ro).max()), "tolerance": 1e-5}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
