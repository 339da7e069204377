"""Benchmark of the FAVOR# hot path: one step = statistics -> fit -> prep -> featurize ->
contraction over one batch of synthetic input.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3+cfg3b|cfg2|cfg3|cfg3b|cfg5]
  python bench.py --impl reference ...     times the fp64 CPU checker instead (bounded sample)

The default workload is the pair of L = 8192, d = 64, M = 256 configurations, causal (cfg3) and
bidirectional (cfg3b): a step is one pass of each, `value` counts the tokens of both.  One step is in
flight at a time (--streams S > 1 keeps S independent steps in flight and reports that figure under
"overlapped", never as the headline).
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

import numpy as np  # noqa: E402

METRIC = "FAVOR# attention tokens/sec/GPU and % of roofline (fwd, bidirectional + causal)"
UNIT = "tokens/s"
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}      # dense bf16 and HBM3e figures of the data sheet
NOT_ATTEND = ("stats_kernel", "tc_stats_kernel", "fit_kernel")


def algorithmic_work(w):
    """Per step, over all (batch, head) units: flops and HBM bytes of the attend stage counted on
    the method's own sizes (no padding, no L^2 work), and the exponentials."""
    units = w.B * w.H
    L, d, dv, M = w.L, w.d, w.dv, w.M
    feat = 2 * 2 * L * d * M                       # X W^T for queries and keys
    if w.variant == "aderf":
        feat += 2 * 2 * L * d * d                  # dense x^T C x per token
    contr = 2 * 2 * L * M * (dv + 1)               # S^T [V|1] and P (S^T [V|1])
    if w.causal:
        contr += L * w.chunk * M + L * w.chunk * (dv + 1)   # triangular halves of the in-chunk products
    es = 2 if w.dtype == "bf16" else 4
    bytes_ = (2 * L * d + 2 * L * dv) * es
    return {"flops": units * (feat + contr), "bytes": units * bytes_, "exps": units * 2 * L * M}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) during the timed region."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag = index, [], set(), False
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def result(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def physical_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def oracle_units(w, Q, K, V, Om, units):
    """The checker's whole path for the given (b, h) units; returns seconds."""
    from oracle import favor_sharp as fs
    t0 = time.perf_counter()
    for u in units:
        b, h = divmod(u, w.H)
        p = fs.fit_params(Q[b, h], K[b, h], w.variant)
        if not w.causal:
            fs.favor_sharp_attention(Q[b, h], K[b, h], V[b, h], Om, p, causal=False)
        else:
            P, S = fs.features_pair(Q[b, h].astype(np.float64), K[b, h].astype(np.float64), Om, p)
            fs.attend_causal_recurrent(P, S, V[b, h])
    return time.perf_counter() - t0


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def workload_list(name):
    from paper_2302_00787_b200 import workloads as wl
    return [wl.WORKLOADS[n] for n in name.split("+")]


def config_of(ws):
    cfg = {"workload": " + ".join(f"{w.name} ({'causal' if w.causal else 'bidirectional'} {w.variant}, B{w.B} H{w.H} L{w.L} "
                                  f"d{w.d} dv{w.dv} M{w.M}{', chunk ' + str(w.chunk) if w.causal else ''})" for w in ws)}
    return cfg


def run_reference(args, ws):
    """The fp64 CPU checker as it stands, on host cores; each step is a bounded sample of every workload."""
    from paper_2302_00787_b200 import workloads as wl
    from paper_2302_00787_b200.sharding import env_rank_world
    rank, _, world = env_rank_world()
    if rank != 0:
        return
    t, tokens, samples = 0.0, 0.0, []
    for w in ws:
        n_units = max(1, min(w.B * w.H, args.ref_units))
        wsmall = w.scaled(B=1, H=n_units)
        Q, K, V = wl.make_qkv(wsmall)
        Om = wl.make_omega(wsmall)
        for _ in range(args.warmup):
            oracle_units(wsmall, Q, K, V, Om, range(1))
        for _ in range(args.steps):
            t += oracle_units(wsmall, Q, K, V, Om, range(n_units))
        tokens += args.steps * n_units * w.L / w.H          # tokens = B * L: a unit is 1/H of a sequence
        samples.append(f"{n_units} of {w.B * w.H} (batch, head) units of {w.name}")
    value = tokens / t
    cores = cpu_threads()
    sample = "; ".join(samples) + " per step (statistics, fit, features, contraction)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(ws),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def rank_setup(n_gpus_asked):
    """(rank, local_rank, world) of this process.  Launched by hand with --gpus N > 1 and no WORLD_SIZE in the
    environment, the caller re-executes itself under torch.distributed.run (see relaunch_if_needed)."""
    from paper_2302_00787_b200.sharding import env_rank_world
    rank, local_rank, world = env_rank_world()
    if "WORLD_SIZE" in os.environ and n_gpus_asked not in (world, 1) and rank == 0:
        print(f"bench.py: --gpus {n_gpus_asked} but WORLD_SIZE={world}; using {world}", file=sys.stderr)
    return rank, local_rank, world


def relaunch_if_needed(args):
    """`python bench.py --gpus N` (N > 1) outside a launcher: start N ranks on this node and pass their output on."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ or args.impl == "reference":
        return False
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


class Runner:
    """One workload resident on the device: `buffers` independent input draws (rotated step by step so that a
    step's inputs are cold in L2), one context with its own scratch, statistics, parameters and output."""

    def __init__(self, w, args, dev, local_rank, seed_shift):
        import torch
        from paper_2302_00787_b200 import binding as fb
        from paper_2302_00787_b200 import workloads as wl
        self.w, self.dev = w, dev
        self.td = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        wr = w.scaled(seed=w.seed + seed_shift)
        self.sets, self.host_set = [], None
        for i in range(args.buffers):
            Q, K, V = wl.make_qkv(wr.scaled(seed=wr.seed + i))
            if i == 0:
                self.host_set = (Q, K, V)
            self.sets.append(tuple(torch.from_numpy(a).to(dev).to(self.td) for a in (Q, K, V)))
        self.Om = wl.make_omega(wr)
        self.dOm = torch.from_numpy(self.Om).to(dev)
        G = w.B * w.H
        self.ctx = fb.Context(local_rank, stream=torch.cuda.current_stream(dev))
        self.ctx.set_impl({"auto": fb.IMPL_AUTO, "simt": fb.IMPL_SIMT, "tensor": fb.IMPL_TENSOR}[args.kernel_impl])
        self.st = torch.empty(G, fb.stats_doubles(w.d), dtype=torch.float64, device=dev)
        self.pr = torch.empty(G, fb.params_doubles(w.d), dtype=torch.float64, device=dev)
        self.Y = torch.empty(w.B, w.H, w.L, w.dv, dtype=self.td, device=dev)

    def step(self, i):
        self.stats(i)
        self.ctx.fsharp_fit_params(self.st, self.w.d, self.w.variant, out=self.pr)
        self.attend(i)

    def stats(self, i):
        dQ, dK, _ = self.sets[i % len(self.sets)]
        self.ctx.fsharp_stats(dQ, dK, out=self.st)

    def attend(self, i):
        dQ, dK, dV = self.sets[i % len(self.sets)]
        w = self.w
        self.ctx.fsharp_attend(dQ, dK, dV, self.dOm, self.pr, causal=w.causal, chunk=w.chunk, out=self.Y)

    def host_buffers(self):
        import torch
        hQ, hK, hV = (torch.from_numpy(a).to(self.td).pin_memory() for a in self.host_set)
        hOm = torch.from_numpy(self.Om).pin_memory()
        hY = torch.empty(self.w.B, self.w.H, self.w.L, self.w.dv, dtype=self.td).pin_memory()
        return hQ, hK, hV, hOm, hY


def backward_flops(w):
    """Multiply-adds x 2 of the backward pass as the kernels issue them (Section 2.2 differentiated; the header of
    csrc/backward.cu lists the products): features of both sides, the two key- / query-side sums, numerators and
    normalisers, the gradients of the features, dV, and the two products back to Q and K; causal adds the masked
    blocks of each chunk (half of a full block each)."""
    L, d, dv, M, N = w.L, w.d, w.dv, w.M, w.dv + 1
    per = 2 * (2 * L * M * d) + 2 * (2 * L * M * N) + 3 * (2 * L * M * N) + 2 * L * M * dv + 2 * (2 * L * M * d + 2 * L * d * d)
    if w.causal:
        C = w.chunk
        per += L * C * (M + N) + L * C * (N + 2 * M + dv)
    return float(per * w.B * w.H)


def backward_leg(runners, sm_count, sm_mhz):
    """fsharp_attend_backward on the bench workloads: CUDA-event time of the call (its kernels run on the fp32 cores),
    against the fp32 multiply-add peak: SMs x 128 lanes x 2 flops x the SM clock seen under load."""
    import torch
    res = {}
    peak = sm_count * 128 * 2 * sm_mhz * 1e6 / 1e12
    for r in runners:
        w = r.w
        dQ, dK, dV = r.sets[0]
        g = torch.Generator(device=dQ.device).manual_seed(w.seed + 99)
        dY = torch.randn(w.B, w.H, w.L, w.dv, generator=g, device=dQ.device, dtype=torch.float32).to(r.td)
        call = lambda: r.ctx.fsharp_attend_backward(dQ, dK, dV, dY, r.dOm, r.pr, causal=w.causal, chunk=w.chunk)
        for _ in range(2):
            call()
        torch.cuda.synchronize()
        n = 3
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            grads = call()
        e1.record()
        torch.cuda.synchronize()
        assert r.ctx.status() == 0
        ms = e0.elapsed_time(e1) / n
        fl = backward_flops(w)
        res[w.name] = {"ms": ms, "tokens_per_s": w.B * w.L / (ms * 1e-3), "gflop": fl / 1e9,
                       "roofline": {"bound": "alu", "achieved": fl / (ms * 1e-3) / 1e12, "peak": peak, "unit": "TFLOP/s",
                                    "frac": fl / (ms * 1e-3) / 1e12 / peak},
                       "finite": bool(all(torch.isfinite(t.float()).all().item() for t in grads))}
        del grads, dY
    return res


# DRAM bytes per launch (read + write) from the ncu captures summarised under profiles/ (same kernels, same
# workload); an entry is dropped when its kernel changes.
NCU_TRAFFIC = {("cfg3", "tc_causal_kernel"): 194.3e6,      # 162.3 MB read + 32.1 MB written (Y stays partly in L2)
               ("cfg3b", "tc_kv_kernel"): 108.4e6, ("cfg3b", "tc_out_kernel"): 70.5e6}


def kernel_flops(name, w, work):
    """Algorithmic flops of one launch of an attention kernel (its share of algorithmic_work)."""
    units = w.B * w.H
    L, d, dv, M = w.L, w.d, w.dv, w.M
    one_side = (2 * L * d * M + 2 * L * M * (dv + 1)) * units
    if name == "tc_causal_kernel":         # everything but the per-key quadratic term (tc_rowterm_kernel)
        return work["flops"] - (2 * 2 * L * d * d * units if w.variant == "aderf" else 0)
    if name in ("tc_kv_kernel", "tc_out_kernel") and not w.causal:
        return one_side
    return None


def run_pairs(args):
    """The variance-study batch (--workload cfg4): for each of the four parameterisations, R draws of estimates for
    every pair, the closed-form variances and the two pooled relative variances.  One line, in pairs/s."""
    import torch
    from paper_2302_00787_b200 import binding as fb
    from paper_2302_00787_b200 import workloads as wl
    pw = wl.PAIR_WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    X, Y = wl.make_pairs(pw.npairs, pw.d, pw.seed)
    Om = wl.make_pair_omegas(pw)
    dX, dY, dOm = (torch.from_numpy(a).to(dev) for a in (X, Y, Om))
    ctx = fb.Context(0)
    st = ctx.fsharp_stats(dX.view(1, 1, pw.npairs, pw.d), dY.view(1, 1, pw.npairs, pw.d))
    prs = [ctx.fsharp_fit_params(st, pw.d, v) for v in pw.variants]
    est = torch.empty(pw.R, pw.npairs, dtype=torch.float32, device=dev)
    pooled = {}

    def step():
        for v, pr in zip(pw.variants, prs):
            pooled[v] = ctx.fsharp_pair_estimate(dX, dY, dOm, pr, want_pooled=True, est=est)[2]

    steps, warm = max(1, min(args.steps, 10)), 3
    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    assert ctx.status() == 0
    sampler = ClockSampler(physical_index(0))
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = ctx.launch_count()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    launches = ctx.launch_count() - n0
    ctx.set_timing(True)
    step()
    kern = ctx.read_timing()
    ctx.set_timing(False)
    sampler.stop_flag = True
    sampler.join(timeout=2)
    nv = len(pw.variants)
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    flops = nv * pw.R * pw.npairs * 2 * (2 * pw.M * pw.d)            # both sides' w^T B x per pair, draw and variant
    peak = 128 * 2 * sm_count * 1965e6 / 1e12                           # fp32: 128 multiply-adds per clock and SM
    t_k = kern["pairs_kernel"][0] / kern["pairs_kernel"][1] * 1e-3
    out = {"metric": "kernel estimates for (x, y) pairs with empirical and closed-form variance", "value": pw.npairs / (ms * 1e-3),
           "unit": "pairs/s", "n_gpus": 1, "steps": steps, "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": f"{pw.name}: {pw.npairs} pairs, d {pw.d}, M {pw.M} orthogonal features, R {pw.R} draws, "
                                  f"parameterisations {', '.join(pw.variants)} (a step covers all of them)"},
           "clocks": sampler.result(), "gpu_launches": launches,
           "roofline": {"kernel": "pairs_kernel", "bound": "alu", "achieved": flops / nv / t_k / 1e12, "peak": peak, "unit": "TFLOP/s",
                        "frac": flops / nv / t_k / 1e12 / peak, "traffic": None,
                        "peak_source": "128 fp32 multiply-adds per clock and SM x SMs x 1965 MHz"},
           "kernels": {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1]} for k, v in kern.items()},
           "pooled_relative_variance": {v: {"empirical": float(pooled[v][0]), "closed_form": float(pooled[v][1])} for v in pw.variants}}
    if not args.no_cpu_baseline:
        from oracle import favor_sharp as fs
        n = 4096
        pr0 = fb.unpack_params(prs[0].cpu().numpy()[0], pw.d)
        t0 = time.perf_counter()
        for r in range(2):
            fs.pair_estimate(X[:n], Y[:n], Om[r], pr0)
        t_est = time.perf_counter() - t0
        t0 = time.perf_counter()
        fs.pair_closed_form_variance(X[:256], Y[:256], pr0, pw.M)
        t_var = time.perf_counter() - t0
        # scaled to one step: every pair gets R draws of estimates and one closed-form variance per parameterisation
        per_est, per_var = t_est / (2 * n), t_var / 256
        out["cpu_baseline"] = {"value": 1.0 / (nv * (pw.R * per_est + per_var)), "unit": "pairs/s", "cores": cpu_threads(), "kind": "oracle",
                               "sample": f"{n} pairs x 2 draws of estimates and 256 closed-form variances of one parameterisation, "
                                         "scaled to all draws and parameterisations"}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="cfg3+cfg3b")
    ap.add_argument("--ref-units", type=int, default=1)
    ap.add_argument("--buffers", type=int, default=3, help="input sets rotated so that a step's inputs are cold in L2")
    ap.add_argument("--cpu-baseline-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--backward", action="store_true",
                    help="also time fsharp_attend_backward on the workloads (fp32 kernels; a few GB of scratch)")
    ap.add_argument("--fit-per-workload", action="store_true",
                    help="one fit launch per workload instead of one launch over the groups of all workloads of a step")
    ap.add_argument("--kernel-impl", default="auto", choices=["auto", "simt", "tensor"])
    args = ap.parse_args()

    if args.workload == "cfg4":
        run_pairs(args)
        return
    ws = workload_list(args.workload)
    if args.impl == "reference":
        run_reference(args, ws)
        return
    relaunch_if_needed(args)

    import torch
    import torch.distributed as dist
    from paper_2302_00787_b200.sharding import max_over_ranks, rank_seed

    rank, local_rank, world = rank_setup(args.gpus)
    if args.warmup < 3:
        args.warmup = 3
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    # weak scaling: every rank runs the whole workload on a draw of its own; no data-path collective
    runners = [Runner(w, args, dev, local_rank, rank_seed(0, rank)) for w in ws]
    stream = torch.cuda.current_stream(dev)
    # The closed-form fit runs one block per parameter group and is bound by the latency of its factorisations, not by
    # the number of groups: the workloads of a step that share (d, variant) are fitted by ONE launch over all their
    # groups.  Their statistics and parameters then live in one buffer each, of which every workload holds a slice.
    joint_fit = (not args.fit_per_workload and len(runners) > 1
                 and len({(r.w.d, r.w.variant) for r in runners}) == 1)
    if joint_fit:
        from paper_2302_00787_b200 import binding as fb
        groups = [r.st.shape[0] for r in runners]
        st_all = torch.empty(sum(groups), fb.stats_doubles(ws[0].d), dtype=torch.float64, device=dev)
        pr_all = torch.empty(sum(groups), fb.params_doubles(ws[0].d), dtype=torch.float64, device=dev)
        g0 = 0
        for r, g in zip(runners, groups):
            r.st, r.pr = st_all[g0:g0 + g], pr_all[g0:g0 + g]
            g0 += g
    torch.cuda.synchronize()

    def step(i):
        if not joint_fit:
            for r in runners:
                r.step(i)
            return
        for r in runners:
            r.stats(i)
        runners[0].ctx.fsharp_fit_params(st_all, ws[0].d, ws[0].variant, out=pr_all)
        for r in runners:
            r.attend(i)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    codes = [r.ctx.status() for r in runners]
    assert all(c == 0 for c in codes), f"device status after warm-up: {codes}"
    sampler = ClockSampler(physical_index(local_rank))
    barrier()
    sampler.start()
    n0 = sum(r.ctx.launch_count() for r in runners)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = sum(r.ctx.launch_count() for r in runners) - n0
    # the steps once more with an event pair around every launch: per-kernel device time
    per_launch = max(1, launches // args.steps)
    ksteps = max(1, min(args.steps, 2048 // per_launch))
    for r in runners:
        r.ctx.set_timing(True)
    for i in range(ksteps):
        step(i)
    per_kernel = [r.ctx.read_timing() for r in runners]
    for r in runners:
        r.ctx.set_timing(False)
    # the attend call alone (parameters given: prep + features + contraction), one event pair around each call; the
    # host runs ahead of the device, so a pair brackets device time only (no per-kernel event records inside)
    attend_direct_ms = []
    for r in runners:
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ksteps)]
        torch.cuda.synchronize()
        for i, (a0, a1) in enumerate(pairs):
            dQ, dK, dV = r.sets[i % len(r.sets)]
            a0.record(stream)
            r.ctx.fsharp_attend(dQ, dK, dV, r.dOm, r.pr, causal=r.w.causal, chunk=r.w.chunk, out=r.Y)
            a1.record(stream)
        torch.cuda.synchronize()
        ts = sorted(a0.elapsed_time(a1) for a0, a1 in pairs)
        attend_direct_ms.append(ts[len(ts) // 2])
    # and every workload's steps by themselves
    alone_ms = []
    for r in runners:
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a0.record(stream)
        for i in range(ksteps):
            r.step(i)
        a1.record(stream)
        torch.cuda.synchronize()
        alone_ms.append(a0.elapsed_time(a1) / ksteps)
    sampler.stop_flag = True
    sampler.join(timeout=2)
    codes = [r.ctx.status() for r in runners]
    assert all(c == 0 for c in codes), f"device status after the timed region: {codes}"
    ms = max_over_ranks(ms, dev)

    # end to end through the host-buffer entry point (pinned host memory; copies inside the timing)
    e2e = None
    if not args.no_e2e:
        bufs = [r.host_buffers() for r in runners]
        n_e2e = max(2, min(args.steps, 10))

        def host_step():
            for r, (hQ, hK, hV, hOm, hY) in zip(runners, bufs):
                # returns when the step's output is in host memory
                r.ctx.fsharp_forward_host(hQ, hK, hV, hOm, r.w.variant, causal=r.w.causal, chunk=r.w.chunk, out=hY)

        for _ in range(3):
            host_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            host_step()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0), dev)
        h2d = sum((hQ.numel() + hK.numel() + hV.numel()) * hQ.element_size() + hOm.numel() * 4 for hQ, hK, hV, hOm, _ in bufs)
        d2h = sum(hY.numel() * hY.element_size() for *_, hY in bufs)
        e2e = (e2e_ms, n_e2e, h2d, d2h)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens_per_step = world * sum(w.B * w.L for w in ws)
    value = tokens_per_step * args.steps / (ms * 1e-3)
    peaks = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_burst": 1590.0, "source": "fallback", "sm_max_mhz": 1965.0}
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        j = json.load(open(pk))
        peaks = {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops_sustained"], "bf16_tflops_burst": j["bf16_tflops"],
                 "source": "measured (sustained bf16: the kernels are timed inside a long step)", "sm_max_mhz": j.get("sm_max_mhz", 1965.0)}
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count

    per_workload, attend_ms_total, roof_ms_total, roof_nominal_total, exp_ms_total = {}, 0.0, 0.0, 0.0, 0.0
    dominant = None
    for r, pkern, alone, attend_ms in zip(runners, per_kernel, alone_ms, attend_direct_ms):
        w = r.w
        work = algorithmic_work(w)
        kernels = {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1] / ksteps, "ms_per_step": v[0] / ksteps}
                   for k, v in sorted(pkern.items(), key=lambda kv: -kv[1][0])}
        attend_kernels_ms = sum(v["ms_per_step"] for k, v in kernels.items() if k not in NOT_ATTEND)
        t_roof = max(work["flops"] / (peaks["bf16_tflops"] * 1e12), work["bytes"] / (peaks["hbm_gbs"] * 1e9)) * 1e3
        t_nom = max(work["flops"] / (NOMINAL["bf16_tflops"] * 1e12), work["bytes"] / (NOMINAL["hbm_gbs"] * 1e9)) * 1e3
        exp_ms = work["exps"] / (16.0 * sm_count * peaks["sm_max_mhz"] * 1e6) * 1e3
        attend_ms_total += attend_ms
        roof_ms_total += t_roof
        roof_nominal_total += t_nom
        exp_ms_total += exp_ms
        per_workload[w.name] = {
            "ms_per_step_alone": alone, "tokens_per_s_alone": w.B * w.L / (alone * 1e-3),
            "attend": {"ms": attend_ms, "tokens_per_s": w.B * w.L / (attend_ms * 1e-3),
                       "algorithmic_tflops": work["flops"] / (attend_ms * 1e-3) / 1e12,
                       "algorithmic_gbs": work["bytes"] / (attend_ms * 1e-3) / 1e9,
                       "gexp_per_s": work["exps"] / (attend_ms * 1e-3) / 1e9,
                       "roofline_ms": t_roof, "roofline_frac": t_roof / attend_ms,
                       "roofline_frac_nominal": t_nom / attend_ms,
                       # a third ceiling: one exponential per feature on the special-function unit (16 per clock and SM)
                       "exp_bound_ms": exp_ms,
                       # the same stage as the sum of its kernels, each bracketed by its own pair of event records
                       "ms_sum_of_kernels": attend_kernels_ms},
            "stats_ms": sum(v["ms_per_step"] for k, v in kernels.items() if k in ("stats_kernel", "tc_stats_kernel")),
            "fit_ms": kernels.get("fit_kernel", {}).get("ms_per_step", 0.0),
            "fit_sweeps": float(r.pr[:, 5 * w.d * w.d + 3].mean().item()),
            "algorithmic": work, "kernels": kernels}
        for k, v in kernels.items():
            if k in NOT_ATTEND:
                continue
            if dominant is None or v["ms_per_step"] > dominant[2]["ms_per_step"]:
                dominant = (w, k, v, work)

    dw, dk, dv_, dwork = dominant
    fl = kernel_flops(dk, dw, dwork)
    t = dv_["ms_per_launch"] * 1e-3
    if fl is not None:
        ach = fl / t / 1e12
        roof = {"kernel": dk, "workload": dw.name, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops"], "frac_nominal": ach / NOMINAL["bf16_tflops"],
                "traffic": NCU_TRAFFIC.get((dw.name, dk)), "peak_source": peaks["source"], "us_per_launch": t * 1e6}
    else:
        by = dwork["bytes"] / max(dv_["launches_per_step"], 1.0)
        ach = by / t / 1e9
        roof = {"kernel": dk, "workload": dw.name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL["hbm_gbs"],
                "traffic": NCU_TRAFFIC.get((dw.name, dk)), "peak_source": peaks["source"], "us_per_launch": t * 1e6}

    cfg = config_of(ws)
    cfg.update({"kernel_impl": args.kernel_impl, "steps_in_flight": 1,
                "l2": f"inputs rotate over {args.buffers} resident sets per workload "
                      f"({args.buffers * algorithmic_work(ws[0])['bytes'] / 1e6:.0f} MB > 126 MB L2)",
                "step": ("stats per workload, one fit launch over the parameter groups of all workloads, then prep + featurize + "
                         "contraction per workload" if joint_fit else "per workload: stats + fit + prep + featurize + contraction")})
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": ws[0].dtype, "data": "synthetic", "config": cfg,
        "clocks": sampler.result(),
        "gpu_launches": launches,
        "roofline": roof,
        "attend": {"ms": attend_ms_total, "tokens_per_s": sum(w.B * w.L for w in ws) / (attend_ms_total * 1e-3),
                   "roofline_ms": roof_ms_total, "roofline_frac": roof_ms_total / attend_ms_total,
                   "roofline_frac_nominal": roof_nominal_total / attend_ms_total, "exp_bound_ms": exp_ms_total,
                   "peaks": peaks, "nominal_peaks": NOMINAL},
        "workloads": per_workload,
    }
    if joint_fit:
        fk = per_kernel[0].get("fit_kernel")
        out["fit"] = {"launches_per_step": 1, "groups": int(st_all.shape[0]),
                      "ms": fk[0] / fk[1] if fk else None,
                      "note": "one launch fits the groups of all workloads of the step (one block per group); every "
                              "workload's ms_per_step_alone includes a fit launch of its own"}
    if args.backward and world == 1:
        clk = out["clocks"].get("sm_mhz") or out["clocks"].get("sm_max_mhz") or 1965
        out["backward"] = backward_leg(runners, torch.cuda.get_device_properties(dev).multi_processor_count, float(clk))
    if e2e is not None:
        e2e_ms, n_e2e, h2d, d2h = e2e
        out["e2e"] = {"value": tokens_per_step * n_e2e / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h}
    if not args.no_cpu_baseline:
        n, t_cpu, tok, parts = 0, 0.0, 0.0, []
        budget = args.cpu_baseline_seconds / len(runners)
        for r in runners:
            Q, K, V = r.host_set
            k, tw = 0, 0.0
            while tw < budget and k < r.w.B * r.w.H:
                tw += oracle_units(r.w, Q, K, V, r.Om, [k])
                k += 1
            t_cpu += tw
            tok += k * r.w.L / r.w.H
            parts.append(f"{k} of {r.w.B * r.w.H} (batch, head) units of {r.w.name}")
        out["cpu_baseline"] = {"value": tok / t_cpu, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                               "sample": "; ".join(parts) + ": statistics, fit, features, contraction"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
