#!/usr/bin/env python
"""Benchmark of the delayed rotated-Adam step (one step = one br_step over the whole layer set).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl reference]

Prints ONE JSON line.  `value` is whole-job parameters/s (steps/s x parameters of the layer set)
with gradients resident in HBM; `e2e` is the same metric through the C-ABI with the gradients in
pinned host memory (host->device copy and a device->host read inside the timed region).
With N > 1 every rank runs an independent replica of the workload (the path has no exchange
step); times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import get_workload  # noqa: E402
from workloads.configs import GEOM_BI, GEOM_NONE, GEOM_UNI, SRC_SECOND  # noqa: E402

# profiles/k_tc_gemm_c5_1layer.md: 11.38e9 B of DRAM traffic for the five launches of one step, which
# execute 6.395e12 flop
NCU_DRAM_BYTES_PER_EXECUTED_FLOP = 11.38e9 / 6.395e12

METRIC = "rotated_adam_params_per_sec"
UNIT = "params/s"


# ---------------------------------------------------------------------------------------------
def algorithmic_flops_per_step(w) -> float:
    """Contraction work the method itself prescribes per step (Alg. 1 (rotation, second moment, weight update) and the factor
    EMAs of Alg. 2): bilateral/2nd 8mn(m+n); one-sided on side s: 8 s^2 max (2nd) or 6 s^2 max (1st)."""
    f = 0.0
    for l in w.layers:
        m, n = l.m, l.n
        if l.geom == GEOM_BI:
            f += (8.0 if l.src == SRC_SECOND else 6.0) * m * n * (m + n)
        elif l.geom == GEOM_UNI:
            s, b = min(m, n), max(m, n)
            f += (8.0 if l.src == SRC_SECOND else 6.0) * s * s * b
    return f


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tf_burst=d["bf16_tflops"], tf_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured (MEASURED_PEAKS.json)")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "200", "-i", str(index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v == "Active":
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
class DeviceGradients:
    """Synthetic gradients generated on the device with the value structure of the workload
    (throughput runs only; parity runs use the CPU streams of workloads.gradients).  The signal
    factors of a low-rank-plus-noise layer are drawn once, the noise is drawn afresh by every call of
    `fresh()`, as the workload prescribes: the factor EMAs then have full rank and the basis refresh
    sees the conditioning of a real stream (a refresh takes device-side decisions that depend on it)."""

    def __init__(self, w, device, torch):
        self.w, self.device, self.torch = w, device, torch
        self.gen = torch.Generator(device=device)
        self.gen.manual_seed(1000003 * (w.seed + 1))
        self.factors = []
        dt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
        self.grads = [torch.empty(l.m, l.n, device=device, dtype=dt) for l in w.layers]
        if w.grad_kind == "lowrank_noise":
            for l in w.layers:
                self.factors.append((torch.randn(l.m, w.grad_rank, device=device, generator=self.gen),
                                     torch.randn(l.n, w.grad_rank, device=device, generator=self.gen)))
        self.fresh()

    def fresh(self):
        torch, w = self.torch, self.w
        for i, l in enumerate(w.layers):
            if w.grad_kind == "lowrank_noise":
                A, B = self.factors[i]
                x = torch.randn(l.m, l.n, device=self.device, generator=self.gen).mul_(w.grad_scale)
                x.addmm_(A, B.t())
            elif w.grad_kind == "student_t":
                z = torch.randn(l.m, l.n, device=self.device, generator=self.gen)
                c = torch.zeros(l.m, l.n, device=self.device)
                for _ in range(3):
                    c.addcmul_(*(2 * [torch.randn(l.m, l.n, device=self.device, generator=self.gen)]))
                x = z.div_(c.div_(3.0).sqrt_()).mul_(w.grad_scale)
            else:
                x = torch.randn(l.m, l.n, device=self.device, generator=self.gen).mul_(w.grad_scale)
            self.grads[i].copy_(x)
            del x
        return self.grads


def max_over_ranks(values, world, device, torch):
    """Times of a multi-rank run are the maximum over the ranks (every rank runs the same replica)."""
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def replica_value(n_params, world, ms_per_step):
    """Whole-job parameters per second of `world` independent replicas that each take ms_per_step."""
    return world * n_params / (ms_per_step / 1e3)


def fit_tau(w_name, n_layers, tau_req, gemm_prec, free_bytes, margin, br):
    """Largest ring depth <= tau_req whose state fits the device (ring bytes are linear in tau)."""
    def total(tau):
        w = get_workload(w_name, n_layers=n_layers, tau=tau)
        descs = [br.BrLayerDesc(m=l.m, n=l.n, geom=l.geom, src=l.src, grad_dtype=br.BR_BF16 if w.grad_dtype == "bf16" else br.BR_F32,
                                tau_max=l.tau_max, freq=0, reserved=0, weight=0) for l in w.layers]
        hp = br.BrHparams(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, weight_decay=0.0, beta_factor=-1.0, freq=w.freq,
                          power_iters=1, accum=0, gemm_prec=gemm_prec, flags=0, clip_norm=0.0, scratch_limit_bytes=0)
        return br.br_state_bytes(descs, hp)[0]
    tau = tau_req
    while tau > 1 and total(tau) > free_bytes - margin:
        tau -= 1
    return tau, total(tau)


# ---------------------------------------------------------------------------------------------
def cpu_oracle_refresh(w, shapes):
    """Seconds the oracle's Power() takes for the bases of the given layer shapes, per refresh.  One
    Power(F, Q) (float64 product + QR, the library QR routine as its step: the written-out Householder
    form takes about a minute at order 2560) is timed at the smallest distinct order; larger orders are
    composed by k^3.  Returns (seconds, description)."""
    import numpy as np
    from oracle import br_oracle as O
    orders = []
    for (m, n, geom, src) in shapes:
        if geom == GEOM_BI or (geom == GEOM_UNI and m <= n):
            orders.append(m)
        if geom == GEOM_BI or (geom == GEOM_UNI and m > n):
            orders.append(n)
    if not orders:
        return 0.0, "no rotated side"
    k0 = min(orders)
    rng = np.random.default_rng(1)
    X = rng.standard_normal((k0, 2 * k0))
    F = X @ X.T / (2 * k0)
    t0 = time.perf_counter()
    O.power(F, np.eye(k0), qr=O.qr_pos_lapack)
    t_k0 = time.perf_counter() - t0
    total = sum(t_k0 * (k / k0) ** 3 for k in orders)
    return total, f"Power() timed at order {k0} ({t_k0:.2f} s), orders {sorted(set(orders))} composed by k^3"


def cpu_oracle_sample(w, shapes, reps=1):
    """Time the float64 oracle (as it stands) on one steady step of each given layer shape."""
    import numpy as np
    from oracle import br_oracle as O
    from dataclasses import replace
    import threadpoolctl
    np.ones((256, 256)) @ np.ones((256, 256))
    total_t, total_params = 0.0, 0
    for (m, n, geom, src) in shapes:
        rng = np.random.default_rng(0)
        lay = O.OracleLayer(np.zeros((m, n)), geom, src, 0)
        orc = O.Oracle([lay], O.Hyper(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, freq=10 ** 9))
        g = rng.standard_normal((m, n))
        best = None
        for _ in range(reps):
            t0 = time.perf_counter()
            orc.step([g], 0)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        total_t += best
        total_params += m * n
    try:
        threads = max(p["num_threads"] for p in threadpoolctl.threadpool_info() if p.get("user_api") == "blas")
    except Exception:
        threads = len(os.sched_getaffinity(0))
    t_refresh, how = cpu_oracle_refresh(w, shapes)
    amortised = total_t + t_refresh / w.freq
    return total_params / amortised, amortised, threads, dict(step_seconds=total_t, refresh_seconds=t_refresh, refresh=how)


def sample_shapes(w, small: bool):
    """Distinct (m, n, geom, src) of the workload, largest first; `small` keeps only the cheapest."""
    seen = []
    for l in w.layers:
        key = (l.m, l.n, l.geom, l.src)
        if l.geom != GEOM_NONE and key not in seen:
            seen.append(key)
    seen.sort(key=lambda k: k[0] * k[1] * (k[0] + k[1]))
    # bounded: drop shapes whose float64 step is beyond ~1.5e12 flop (e.g. a 32000-row embedding factor)
    seen = [k for k in seen if 8.0 * k[0] * k[1] * (k[0] + k[1]) <= 1.5e12] or seen[:1]
    return seen[:1] if small else seen[:3]


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = get_workload(args.workload)
    shapes = sample_shapes(w, small=True)
    times = []
    for i in range(args.warmup + args.steps):
        v, t, threads, parts = cpu_oracle_sample(w, shapes)
        if i >= args.warmup:
            times.append(t)
    ms = 1e3 * sum(times) / len(times)
    params = sum(m * n for m, n, _, _ in shapes)
    value = params / (ms / 1e3)
    sample = ("one oracle step of a %dx%d matrix of %s + (one Power() of each of its bases)/freq per step; %s; the %s is left out of the sample"
              % (shapes[0][0], shapes[0][1], w.name, parts["refresh"], "embedding" if w.name in ("c4", "c5") else "rest of the layer set"))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def deep_ring_check(args, br, torch, dev, stream, tau_req, gemm_prec, main_steady_ms, main_params, main_tau):
    """The steady step with the ring depth the workload asks for, on the largest decoder depth whose state
    fits it: the work of a step (one ring write, one ring read per parameter) should not depend on the
    depth of the ring, only memory does.  Reported as time per parameter beside the main run's."""
    free0, _ = torch.cuda.mem_get_info(dev)
    n_fit = None
    for n_layers in range((args.layers or 32), 0, -1):
        wt = get_workload(args.workload, n_layers=n_layers, tau=tau_req)
        descs = [br.BrLayerDesc(m=l.m, n=l.n, geom=l.geom, src=l.src, grad_dtype=br.BR_BF16, tau_max=l.tau_max, freq=0,
                                reserved=0, weight=0) for l in wt.layers]
        hp = br.BrHparams(lr=wt.lr, beta1=wt.beta1, beta2=wt.beta2, eps=wt.eps, weight_decay=0.0, beta_factor=-1.0, freq=wt.freq,
                          power_iters=1, accum=0, gemm_prec=gemm_prec, flags=0, clip_norm=0.0, scratch_limit_bytes=0)
        need = br.br_state_bytes(descs, hp)[0] + wt.n_params * (4 + 2 + 4) + (6 << 30)
        if need <= free0:
            n_fit = n_layers
            break
    if n_fit is None:
        return {"error": "no depth fits"}
    wt = get_workload(args.workload, n_layers=n_fit, tau=tau_req)
    weights = [torch.empty(l.m, l.n, device=dev).normal_(0.0, 0.02) for l in wt.layers]
    with torch.cuda.stream(stream):
        gen = DeviceGradients(wt, dev, torch)
        opt = br.BasisRotation.from_workload(wt, weights, stream=stream)
        for _ in range(tau_req + 8):
            opt.step(gen.fresh(), tau_req)
        for _ in range(3):
            opt.refresh_basis(-1)
            for _ in range(4):
                opt.step(gen.fresh(), tau_req)
        steps = 10
        ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
        for k in range(steps):
            gen.fresh()
            ev0[k].record(stream)
            opt.step(gen.grads, tau_req)
            ev1[k].record(stream)
        torch.cuda.synchronize(dev)
        assert opt.sync_status() >= 0
        ms = sum(a.elapsed_time(b) for a, b in zip(ev0, ev1)) / steps
        slot = opt.counters(0)["ring_slot"]
    opt.close()
    return {"decoder_layers": n_fit, "params": wt.n_params, "tau": tau_req, "ms_steady_step": ms, "steps": steps,
            "ps_per_param": 1e9 * ms / wt.n_params, "main_run_ps_per_param": 1e9 * main_steady_ms / main_params,
            "main_run_tau": main_tau, "ring_slot_after": slot,
            "note": "same command, same process: the largest decoder depth whose state fits a uniform ring of the requested depth"}


# ---------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c5")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--layers", type=int, default=None, help="decoder depth override (c4/c5)")
    ap.add_argument("--tau", type=int, default=None, help="ring depth override")
    ap.add_argument("--e2e-steps", type=int, default=12)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--scratch-gib", type=float, default=0.0)
    ap.add_argument("--no-tau-check", action="store_true",
                    help="skip the second, shallower run at the requested ring depth (config.tau32_check)")
    ap.add_argument("--profiler-range", default="", choices=["", "steps", "refresh"],
                    help="call cudaProfilerStart/Stop around the timed steps or the timed refresh (for `ncu --profile-from-start off`)")
    ap.add_argument("--no-refresh", action="store_true",
                    help="profiling captures only: skip the basis refresh (priming and timing); the line is then not a bench value")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2602_03515_b200 as br
    from paper_2602_03515_b200 import build as _build
    _build.build()
    br.load_library()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        # one process per GPU: N > 1 needs a launcher that sets WORLD_SIZE / RANK / LOCAL_RANK
        sys.exit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}; launch N > 1 as "
                 f"`python -m torch.distributed.run --nnodes=1 --nproc-per-node {args.gpus} --master-addr 127.0.0.1 "
                 f"--master-port P bench.py --gpus {args.gpus} ...`")
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    peaks = measured_peaks()

    # ---- workload and memory plan -------------------------------------------------------------
    w0 = get_workload(args.workload, n_layers=args.layers, tau=args.tau)
    gemm_prec = br.BR_GEMM_FP32 if w0.gemm_prec == "f32" else br.BR_GEMM_BF16
    tau_req = w0.tau
    free0, total_mem = torch.cuda.mem_get_info(dev)
    n_params0 = w0.n_params
    gbytes = 2 if w0.grad_dtype == "bf16" else 4
    # caller's weights, two gradient sets (the end-to-end leg double-buffers its uploads) + headroom
    reserve = n_params0 * (4 + 2 * gbytes) + (6 << 30)
    if args.workload in ("c4", "c5"):
        tau, state_bytes = fit_tau(args.workload, args.layers, tau_req, gemm_prec, free0, reserve, br)
        w = get_workload(args.workload, n_layers=args.layers, tau=tau)
    else:
        w, tau = w0, tau_req
        state_bytes = None
    n_params = w.n_params

    weights = [torch.empty(l.m, l.n, device=dev).normal_(0.0, 0.02) for l in w.layers]
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        gen = DeviceGradients(w, dev, torch)
    grads = gen.grads
    opt = br.BasisRotation.from_workload(w, weights, stream=stream,
                                         scratch_limit_bytes=int(args.scratch_gib * 2 ** 30))
    if state_bytes is None:
        state_bytes = opt.state_bytes()[0]

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    with torch.cuda.stream(stream):
        # ---- priming (untimed): fill the ring, apply one update, refresh every basis once -------
        # (eight updates before the first refresh: the factor EMAs must have full rank, which takes
        # ceil(max(m, n) / min(m, n)) gradients; in a real run the first refresh comes at t = freq)
        for _ in range(tau + 8):
            opt.step(gen.fresh(), tau)
        # Three untimed refreshes: the first starts from U = V = I and is ill-conditioned, the second
        # already tracks the factors and leaves that note, the third is the first to take the
        # steady-state form (and captures its launch chains into graphs); the timed one is the fourth.
        if args.no_refresh:
            # profiling aid: no refresh is run, so the bases are set to seeded random orthogonal matrices
            # (with U = V = I the low-order operand halves would be zero: not the data a real step sees)
            gen_q = torch.Generator(device=dev)
            gen_q.manual_seed(1234)
            for li, l in enumerate(w.layers):
                left = l.geom == GEOM_BI or (l.geom == GEOM_UNI and l.m <= l.n)      # Alg. 2: the smaller side
                right = l.geom == GEOM_BI or (l.geom == GEOM_UNI and l.m > l.n)
                for which, k, has in ((br.BR_BUF_U, l.m, left), (br.BR_BUF_V, l.n, right)):
                    if has:
                        q, r = torch.linalg.qr(torch.randn(k, k, device=dev, generator=gen_q))
                        opt.set_state(li, which, q * torch.sign(torch.diagonal(r)))
        else:
            for _ in range(3):
                opt.refresh_basis(-1)
                for _ in range(4):
                    opt.step(gen.fresh(), tau)
        assert opt.sync_status() >= 0
        for _ in range(args.warmup):
            opt.step(gen.fresh(), tau)
        sync_all()

        # ---- timed region: exactly K steps, events on the launching stream -----------------------
        l0, _ = opt.launch_stats()
        sampler = ClockSampler(local)
        # (the gradients of a step are drawn before its first event: generating inputs is not timed)
        ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
        is_refresh = []
        opt.profile(True)      # an event pair around every launch of the library: per-kernel device time of the timed steps
        torch.cuda.nvtx.range_push("timed_steps")      # (lets a profiler pick the timed launches by range)
        if args.profiler_range == "steps":
            torch.cuda.synchronize(dev); torch.cuda.profiler.start()
        for k in range(args.steps):
            gen.fresh()
            ev0[k].record(stream)
            opt.step(grads, tau)
            ev1[k].record(stream)
            is_refresh.append(opt.counters(0)["t"] % w.freq == 0)     # every layer shares tau and freq here
        torch.cuda.nvtx.range_pop()
        opt.profile(False)
        sync_all()
        if args.profiler_range == "steps":
            torch.cuda.profiler.stop()
        clocks = sampler.stop()
        prof = opt.get_profile()
        prof_steps = args.steps
        l1, _ = opt.launch_stats()
        step_ms = [ev0[k].elapsed_time(ev1[k]) for k in range(args.steps)]
        total_ms = sum(step_ms)

        # ---- one full refresh (every layer), timed on its own --------------------------------------
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler_r = ClockSampler(local)
        if args.profiler_range == "refresh":
            torch.cuda.synchronize(dev); torch.cuda.profiler.start()
        r0.record(stream)
        torch.cuda.nvtx.range_push("timed_refresh")
        if not args.no_refresh:
            opt.refresh_basis(-1)
        torch.cuda.nvtx.range_pop()
        r1.record(stream)
        sync_all()
        if args.profiler_range == "refresh":
            torch.cuda.profiler.stop()
        clocks_refresh = sampler_r.stop()
        refresh_ms = r0.elapsed_time(r1)

        assert opt.sync_status() >= 0

    steady = [t for t, r in zip(step_ms, is_refresh) if not r] or step_ms
    steady_ms = sum(steady) / len(steady)
    amortised_ms = steady_ms + refresh_ms / w.freq
    amortised_ms, steady_ms, refresh_ms, raw_ms = max_over_ranks(
        [amortised_ms, steady_ms, refresh_ms, total_ms / args.steps], world, dev, torch)
    value = replica_value(n_params, world, amortised_ms)

    # ---- end to end through the C-ABI with host buffers ------------------------------------------
    e2e = None
    if args.e2e_steps > 0:
        host = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True) for g in grads]
        for h_, g in zip(host, grads):
            h_.copy_(g)
        w_host = [torch.empty(weights[0].shape, dtype=torch.float32, pin_memory=True) for _ in range(2)]
        h2d = sum(h_.numel() * h_.element_size() for h_ in host)
        d2h = w_host[0].numel() * 4 + 4
        # Every step uploads its gradients from pinned host memory and reads a weight matrix back; the
        # status word is read at the end.  The upload of step i + 1 runs on a copy stream, into the other of
        # two device gradient sets, while step i computes (the library has copied a call's gradients into
        # its ring by the time the stream passes that call's work, so a set is free again two steps later);
        # the host waits for the result of step i - 1 while step i runs.
        grads2 = [torch.empty_like(g) for g in grads]
        sets = [grads, grads2]
        copy_stream = torch.cuda.Stream(device=dev)
        up = [torch.cuda.Event(), torch.cuda.Event()]          # upload of a set finished
        used = [torch.cuda.Event(), torch.cuda.Event()]        # the step that read a set has been passed
        done = [torch.cuda.Event(), torch.cuda.Event()]        # the result of a step has reached the host

        def upload(i):
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(used[i % 2])
                for h_, g in zip(host, sets[i % 2]):
                    g.copy_(h_, non_blocking=True)
                up[i % 2].record(copy_stream)

        # the leg charges the refresh as (one full refresh)/freq below, so no periodic refresh may fall
        # inside it: if one is due within the next e2e_steps updates, run up to it first (untimed)
        args.e2e_steps = max(1, min(args.e2e_steps, w.freq - 1))
        t_now = opt.counters(0)["t"]
        if (t_now % w.freq) + args.e2e_steps >= w.freq:
            with torch.cuda.stream(stream):
                for _ in range(w.freq - t_now % w.freq):
                    opt.step(gen.fresh(), tau)
        sync_all()
        for ev in used:
            ev.record(stream)
        t0 = time.perf_counter()
        upload(0)
        with torch.cuda.stream(stream):
            for i in range(args.e2e_steps):
                if i + 1 < args.e2e_steps:
                    upload(i + 1)
                stream.wait_event(up[i % 2])
                opt.step(sets[i % 2], tau)
                used[i % 2].record(stream)
                w_host[i % 2].copy_(weights[0], non_blocking=True)
                done[i % 2].record(stream)
                if i >= 1:
                    done[(i - 1) % 2].synchronize()
            st = opt.sync_status()              # waits for the stream and reads the status word back
            assert st >= 0
        sync_all()
        e2e_ms = 1e3 * (time.perf_counter() - t0) / args.e2e_steps + refresh_ms / w.freq
        e2e_ms = max_over_ranks([e2e_ms], world, dev, torch)[0]
        e2e = {"value": replica_value(n_params, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": args.e2e_steps,
               "note": "the step's inputs (every layer's gradient) are uploaded from pinned host memory every step; its result, the updated "
                       "weights, stays on the device where the caller's model owns it -- read back per step are one updated weight "
                       "matrix (%d x %d fp32) and, at the end, the status word" % tuple(weights[0].shape)}
        del host, grads2

    # ---- rooflines -------------------------------------------------------------------------------
    alg_flops = algorithmic_flops_per_step(w)
    roofline = None
    roofline_elem = None
    if prof["tc_launches"] > 0:
        tc_ms_step = prof["tc_ms"] / prof_steps
        achieved = alg_flops / (tc_ms_step / 1e3) / 1e12
        executed = prof["tc_flops"] / (prof["tc_ms"] / 1e3) / 1e12
        # DRAM bytes per launch: dram__bytes_read+write of an ncu capture of a small case of this
        # workload (profiles/), scaled to this run's launches by executed flop per launch
        traffic = NCU_DRAM_BYTES_PER_EXECUTED_FLOP * prof["tc_flops"] / prof["tc_launches"]
        # achieved / frac: what the tensor pipe executed (9 one-sided products per bilateral matrix, the factor
        # products on upper-triangle tiles only); effective_*: the method's own 8 m n (m + n) over the same time
        roofline = {"bound": "tensor", "kernel": "k_tc_gemm", "achieved": executed, "peak": peaks["tf_sustained"],
                    "unit": "TFLOP/s", "frac": executed / peaks["tf_sustained"], "traffic": traffic,
                    "traffic_source": "ncu capture of the 1-layer case (profiles/k_tc_gemm_c5_1layer.md), scaled by executed flop per launch",
                    "effective_tflops": achieved, "effective_frac": achieved / peaks["tf_sustained"],
                    "flops_counted": "executed by the tensor pipe (effective_* counts the algorithmic 8mn(m+n))",
                    "launches_per_step": prof["tc_launches"] / prof_steps, "ms_per_step_in_kernel": tc_ms_step,
                    "avg_launch_ms": prof["tc_ms"] / prof["tc_launches"],
                    "peak_source": peaks["source"] + ", bf16 sustained"}

    # ---- the refresh against its own rooflines ------------------------------------------------------
    roofline_refresh = None
    if not args.no_refresh:
        orders = []
        for l in w.layers:
            if l.geom == GEOM_BI or (l.geom == GEOM_UNI and l.m <= l.n):
                orders.append(l.m)
            if l.geom == GEOM_BI or (l.geom == GEOM_UNI and l.m > l.n):
                orders.append(l.n)
        # per basis of order k: 2 k^3 (the product F Q) + 8/3 k^3 (QR with Q formed); S = 1st adds the factor itself
        ref_flops = sum((2.0 + 8.0 / 3.0) * float(k) ** 3 for k in orders)
        ref_tflops = ref_flops / (refresh_ms / 1e3) / 1e12
        fp64_peak = 148 * 64 * 2 * 1.965e9 / 1e12       # 148 SMs x 64 fp64 FMA per clock (mma.sync.m8n8k4.f64) x 2 x 1.965 GHz
        roofline_refresh = {"bound": "fp64 matrix unit / tensor", "kernel": "k_dgemm + k_chol_inverse + k_tc_gemm (three-term bf16 splits)",
                            "bases": len(orders), "algorithmic_flops": ref_flops, "achieved": ref_tflops, "unit": "TFLOP/s",
                            "peak_fp64_unit": fp64_peak, "frac_of_fp64_unit": ref_tflops / fp64_peak,
                            "peak_bf16_split6": peaks["tf_sustained"] / 6.0, "frac_of_bf16_split6": ref_tflops / (peaks["tf_sustained"] / 6.0),
                            "ms": refresh_ms, "share_of_amortised_step": (refresh_ms / w.freq) / amortised_ms,
                            "peak_source": "fp64: 148 SMs x 64 FMA/clk x 2 x 1.965 GHz (a register-only loop of the instruction reaches 99 % of it); "
                                           "bf16: " + peaks["source"] + " sustained / 6 (six bf16 products per fp32-accurate product)"}

    # ---- element-wise kernel of the path (Eq. (adam) for parameters that are not rotated) ---------------
    # The steady step of a fully rotated layer set runs no element-wise kernel (the moment updates are
    # epilogues of the contractions), so the HBM-bound kernel is timed on its own: one 32000 x 2560
    # matrix with geometry none, 26 B per parameter (g 2, m 8, v 8, w 8), inputs larger than L2.
    try:
        from workloads import LayerSpec
        em, en = 32000, 2560
        we = torch.empty(em, en, device=dev).normal_(0.0, 0.02)
        ge = torch.randn(em, en, device=dev).mul_(1e-3).to(torch.bfloat16)
        with torch.cuda.stream(stream):
            oe = br.BasisRotation([LayerSpec("emb", em, en, GEOM_NONE, SRC_SECOND, 0)], [we], grad_dtype="bf16",
                                  gemm_prec=gemm_prec, stream=stream)
            for _ in range(3):
                oe.step([ge], 0)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 20
            a0.record(stream)
            for _ in range(reps):
                oe.step([ge], 0)
            a1.record(stream)
            torch.cuda.synchronize(dev)
            adam_ms = a0.elapsed_time(a1) / reps
            oe.close()
        gbs = 26.0 * em * en / (adam_ms / 1e3) / 1e9
        roofline_elem = {"bound": "hbm", "kernel": "k_plain_adam", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm"], "traffic": None, "avg_launch_ms": adam_ms,
                         "workload": "32000x2560 matrix, geometry none, bf16 gradient, 26 B/param, 20 launches",
                         "peak_source": peaks["source"] + ", copy bandwidth"}
        del we, ge
    except Exception as ex:                      # the side measurement must not take the bench line down
        roofline_elem = {"error": str(ex)}

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, N = 1 only) -----------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        shapes = sample_shapes(w, small=False)
        v, t, threads, parts = cpu_oracle_sample(w, shapes, reps=3)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": t, **parts,
               "sample": "best of 3 float64 oracle steps of each of " +
                         ", ".join(f"{m}x{n}" for m, n, _, _ in shapes) + f" from {w.name}, plus (one Power() of each of their bases)/freq, "
                         "as the GPU value charges it; the 32000-row embedding is left out of the sample (one float64 step of it is beyond the sample's budget)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": amortised_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if gemm_prec == br.BR_GEMM_BF16 else "f32", "data": "synthetic",
            "steps_per_sec": 1e3 / amortised_ms,
            "ms_steady_step": steady_ms, "ms_full_refresh": refresh_ms, "ms_raw_mean_of_timed_steps": raw_ms,
            "timing": "ms_per_step = mean steady step + (one refresh of every basis)/freq; refresh steps inside the timed region are excluded from the steady mean",
            "config": {"workload": w.name, "layers": len(w.layers), "params": n_params, "geometry": "bilateral+unilateral embedding" if args.workload in ("c4", "c5") else "see workloads/configs.py",
                       "tau": tau, "tau_requested": tau_req, "freq": w.freq, "grad_dtype": w.grad_dtype, "state_bytes": state_bytes,
                       "l2": "inputs larger than L2 (no flush needed)" if n_params * 2 > (126 << 20) else "inputs smaller than L2",
                       "replicas": world, "refresh_skipped_not_a_bench_value": bool(args.no_refresh), "gradients": "device-generated; signal factors fixed per layer, noise drawn afresh before every step (untimed)"},
            "clocks": clocks, "clocks_during_refresh": clocks_refresh, "e2e": e2e, "gpu_launches": int(l1 - l0),
            "roofline": roofline, "roofline_refresh": roofline_refresh, "roofline_elementwise": roofline_elem, "cpu_baseline": cpu,
            "algorithmic_flops_per_step": alg_flops,
        }
    opt.close()
    # ---- the requested ring depth on as many layers as fit it (the full set runs with a shallower ring) ----
    if rank == 0 and world == 1 and args.workload in ("c4", "c5") and tau < tau_req and not args.no_tau_check and not args.no_refresh:
        try:
            del opt, weights, grads, gen
            torch.cuda.empty_cache()
            line["config"]["tau32_check"] = deep_ring_check(args, br, torch, dev, stream, tau_req, gemm_prec, steady_ms, n_params, tau)
        except Exception as ex:                  # the side measurement must not take the bench line down
            line["config"]["tau32_check"] = {"error": str(ex)}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
