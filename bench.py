"""Benchmark of the FAVOR# hot path: one step = statistics -> fit -> prep -> featurize ->
contraction over one batch of synthetic input.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg3b|cfg5]
  python bench.py --impl reference ...     times the fp64 CPU checker instead (bounded sample)
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "FAVOR# attention tokens/sec/GPU and % of roofline (fwd, bidirectional + causal)"
UNIT = "tokens/s"


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
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown if hasattr(nv, "nvmlClocksEventReasonHwSlowdown") else 0x8,
                 "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
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
            time.sleep(0.02)

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
        fs.favor_sharp_attention(Q[b, h], K[b, h], V[b, h], Om, p, causal=False) if not w.causal else \
            fs.attend_causal_recurrent(*fs.features_pair(Q[b, h].astype(np.float64), K[b, h].astype(np.float64), Om, p), V[b, h])
    return time.perf_counter() - t0


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, w):
    """The fp64 CPU checker as it stands, on host cores; each step is a bounded sample."""
    from paper_2302_00787_b200 import workloads as wl
    from paper_2302_00787_b200.sharding import env_rank_world
    rank, _, world = env_rank_world()
    if rank != 0:
        return
    n_units = max(1, min(w.B * w.H, args.ref_units))
    ws = w.scaled(B=1, H=n_units)
    Q, K, V = wl.make_qkv(ws)
    Om = wl.make_omega(ws)
    for _ in range(args.warmup):
        oracle_units(ws, Q, K, V, Om, range(1))
    t = 0.0
    for _ in range(args.steps):
        t += oracle_units(ws, Q, K, V, Om, range(n_units))
    head_tokens = args.steps * n_units * w.L
    value = head_tokens / w.H / t
    cores = cpu_threads()
    sample = f"{n_units} of {w.B * w.H} (batch, head) units of {w.name} per step (statistics, fit, features, contraction)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d": w.d, "dv": w.dv, "M": w.M,
                   "variant": w.variant, "causal": w.causal, "chunk": w.chunk},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--ref-units", type=int, default=2)
    ap.add_argument("--buffers", type=int, default=3, help="input sets rotated so that a step's inputs are cold in L2")
    ap.add_argument("--cpu-baseline-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-impl", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--streams", type=int, default=3,
                    help="steps in flight: step i runs on context i mod S, each context with a stream, scratch and outputs of its own")
    args = ap.parse_args()

    from paper_2302_00787_b200 import workloads as wl
    w = wl.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2302_00787_b200 import binding as fb
    from paper_2302_00787_b200.sharding import env_rank_world, max_over_ranks, rank_seed

    rank, local_rank, world = env_rank_world()
    if args.warmup < 3:
        args.warmup = 3
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    w_rank = w.scaled(seed=rank_seed(w.seed, rank))
    td = torch.bfloat16 if w.dtype == "bf16" else torch.float32

    # inputs: `buffers` independent draws resident in HBM, rotated step by step
    sets = []
    host_set = None
    for i in range(args.buffers):
        wi = w_rank.scaled(seed=w_rank.seed + i)
        Q, K, V = wl.make_qkv(wi)
        if i == 0:
            host_set = (Q, K, V)
        sets.append(tuple(torch.from_numpy(a).to(dev).to(td) for a in (Q, K, V)))
    Om = wl.make_omega(w_rank)
    dOm = torch.from_numpy(Om).to(dev)
    G = w.B * w.H
    # Steps are independent of one another, and the fit keeps one block per group busy (fewer blocks than SMs),
    # so S steps are kept in flight: step i runs on context i mod S.  Every context has a stream, a scratch
    # block, statistics, parameters and an output tensor of its own; nothing is shared but the read-only inputs.
    S = max(1, args.streams)
    main_stream = torch.cuda.current_stream(dev)
    streams = [torch.cuda.Stream(dev) for _ in range(S)] if S > 1 else [main_stream]
    ctxs = [fb.Context(local_rank, stream=s_) for s_ in streams]
    for c in ctxs:
        c.set_impl({"auto": fb.IMPL_AUTO, "simt": fb.IMPL_SIMT, "tensor": fb.IMPL_TENSOR}[args.kernel_impl])
    ctx = ctxs[0]
    sts = [torch.empty(G, fb.stats_doubles(w.d), dtype=torch.float64, device=dev) for _ in ctxs]
    prs = [torch.empty(G, fb.params_doubles(w.d), dtype=torch.float64, device=dev) for _ in ctxs]
    Ys = [torch.empty(w.B, w.H, w.L, w.dv, dtype=td, device=dev) for _ in ctxs]
    pr = prs[0]
    torch.cuda.synchronize()

    def step(i):
        dQ, dK, dV = sets[i % len(sets)]
        c = i % S
        ctxs[c].fsharp_stats(dQ, dK, out=sts[c])
        ctxs[c].fsharp_fit_params(sts[c], w.d, w.variant, out=prs[c])
        ctxs[c].fsharp_attend(dQ, dK, dV, dOm, prs[c], causal=w.causal, chunk=w.chunk, out=Ys[c])

    def fork():
        """The contexts' streams start after everything queued on the timing stream."""
        if S > 1:
            ev = torch.cuda.Event()
            ev.record(main_stream)
            for s_ in streams:
                s_.wait_event(ev)

    def join():
        """The timing stream continues after everything queued on the contexts' streams."""
        if S > 1:
            for s_ in streams:
                ev = torch.cuda.Event()
                ev.record(s_)
                main_stream.wait_event(ev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, S)):
        step(i)
    torch.cuda.synchronize()
    assert all(c.status() == 0 for c in ctxs), "device status after warm-up"
    sampler = ClockSampler(physical_index(local_rank))
    barrier()
    sampler.start()
    n0 = sum(c.launch_count() for c in ctxs)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main_stream)
    fork()
    for i in range(args.steps):
        step(i)
    join()
    e1.record(main_stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = sum(c.launch_count() for c in ctxs) - n0
    # the steps once more, one at a time on one context, with an event pair around every launch:
    # per-kernel device time of a kernel that has the GPU to itself
    ctx.set_timing(True)
    ksteps = max(1, min(args.steps, 4096 // max(1, launches // args.steps)))
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(ksteps):
        step(i * S)
    per_kernel = ctx.read_timing()
    ctx.set_timing(False)
    # and untimed inside, one step at a time: the latency of a step that has the GPU to itself
    torch.cuda.synchronize()
    e2.record(streams[0])
    for i in range(ksteps):
        step(i * S)
    e3.record(streams[0])
    torch.cuda.synchronize()
    serial_ms = e2.elapsed_time(e3) / ksteps
    sampler.stop_flag = True
    sampler.join(timeout=2)
    assert all(c.status() == 0 for c in ctxs), "device status after the timed region"
    ms = max_over_ranks(ms, dev)

    # end to end through the host-buffer entry point (pinned host memory; copies inside the timing)
    hQ, hK, hV = (torch.from_numpy(a).to(td).pin_memory() for a in host_set)
    hOm = torch.from_numpy(Om).pin_memory()
    hYs = [torch.empty(w.B, w.H, w.L, w.dv, dtype=td).pin_memory() for _ in ctxs]
    hY = hYs[0]
    per_thread = max(2, min(args.steps, 20) // S)
    e2e_steps = per_thread * S

    def host_steps(c, n):
        # the call returns when the step's output is in host memory; ctypes releases the interpreter lock meanwhile
        torch.cuda.set_device(local_rank)
        for _ in range(n):
            ctxs[c].fsharp_forward_host(hQ, hK, hV, hOm, w.variant, causal=w.causal, chunk=w.chunk, out=hYs[c])

    for c in range(S):
        host_steps(c, 3)
    barrier()
    # S host threads, one context each: one step's download and compute overlap the next step's upload
    workers = [threading.Thread(target=host_steps, args=(c, per_thread)) for c in range(S)]
    t0 = time.perf_counter()
    for t_ in workers:
        t_.start()
    for t_ in workers:
        t_.join()
    torch.cuda.synchronize()
    e2e_ms = 1e3 * (time.perf_counter() - t0)
    e2e_ms = max_over_ranks(e2e_ms, dev)
    es = 2 if w.dtype == "bf16" else 4
    h2d = (hQ.numel() + hK.numel() + hV.numel()) * es + hOm.numel() * 4
    d2h = hY.numel() * es

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    tokens_per_step = world * w.B * w.L
    value = tokens_per_step * args.steps / (ms * 1e-3)
    work = algorithmic_work(w)
    peaks = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}
    pk = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(pk):
        j = json.load(open(pk))
        peaks = {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops_sustained"], "source": "measured (sustained)",
                 "sm_max_mhz": j.get("sm_max_mhz", 1965.0)}
    # dominant kernel of the step and its roofline
    tot = sum(v[0] for v in per_kernel.values()) or 1.0
    kernels = {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1] / ksteps, "share": v[0] / tot}
               for k, v in sorted(per_kernel.items(), key=lambda kv: -kv[1][0])}
    dom = next(iter(kernels))
    work["fit_sweeps"] = float(pr[:, 5 * w.d * w.d + 3].mean().item())
    peaks["sm_count"] = torch.cuda.get_device_properties(dev).multi_processor_count
    roof = roofline_for(dom, kernels[dom], w, work, peaks)
    attend_ms = sum(v[0] for k, v in per_kernel.items() if k not in ("stats_kernel", "tc_stats_kernel", "fit_kernel")) / ksteps
    t_roof = max(work["flops"] / (peaks["bf16_tflops"] * 1e12), work["bytes"] / (peaks["hbm_gbs"] * 1e9))
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d": w.d, "dv": w.dv, "M": w.M,
                   "variant": w.variant, "causal": w.causal, "chunk": w.chunk, "kernel_impl": args.kernel_impl,
                   "l2": f"inputs rotate over {len(sets)} resident sets ({len(sets) * work['bytes'] / 1e6:.0f} MB > 126 MB L2)",
                   "step": "stats + fit + prep + featurize + contraction",
                   "steps_in_flight": S},
        "ms_per_step_alone": serial_ms,
        "clocks": sampler.result(),
        "e2e": {"value": tokens_per_step * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roof,
        "attend": {"ms": attend_ms, "tokens_per_s": w.B * w.L / (attend_ms * 1e-3),
                   "algorithmic_tflops": work["flops"] / (attend_ms * 1e-3) / 1e12,
                   "algorithmic_gbs": work["bytes"] / (attend_ms * 1e-3) / 1e9,
                   "gexp_per_s": work["exps"] / (attend_ms * 1e-3) / 1e9,
                   "roofline_frac": t_roof * 1e3 / attend_ms, "peaks": peaks},
        "kernels": kernels,
    }
    if not args.no_cpu_baseline:
        Q, K, V = host_set
        n, t = 0, 0.0
        while t < args.cpu_baseline_seconds and n < G:
            t += oracle_units(w, Q, K, V, Om, [n])
            n += 1
        out["cpu_baseline"] = {"value": n * w.L / w.H / t, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                               "sample": f"{n} of {G} (batch, head) units of {w.name}: statistics, fit, features, contraction"}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes per launch (read + write) from the ncu captures summarised under profiles/ (same kernels, same workload);
# an entry is dropped when its kernel changes.
NCU_TRAFFIC = {("cfg2", "fit_kernel"): 4.39e6, ("cfg2", "tc_kv_kernel"): 74.9e6, ("cfg2", "tc_out_kernel"): 48.8e6,
               ("cfg3", "tc_kv_kernel"): 412.4e6, ("cfg3", "tc_causal_out_kernel"): 625.5e6,
               ("cfg3", "tc_featq_kernel"): 195.5e6, ("cfg3", "tc_causal_prefix_kernel"): 178.2e6}


def roofline_for(name, k, w, work, peaks):
    """Roofline entry for the step's dominant kernel.  Algorithmic work per launch:
    tensor-bound kernels carry their share of the attend flops; the rest are judged on bytes."""
    units = w.B * w.H
    L, d, dv, M = w.L, w.d, w.dv, w.M
    es = 2 if w.dtype == "bf16" else 4
    per_launch = 1.0 / max(k["launches_per_step"], 1e-9)
    t = k["ms_per_launch"] * 1e-3
    flops_of = {
        "logits_kernel": 2 * L * d * M * units, "kv_kernel": 2 * L * M * (dv + 1) * units,
        "out_kernel": 2 * L * M * (dv + 1) * units, "scores_kernel": L * w.chunk * M * units if w.causal else 0,
        "tc_kv_kernel": (2 * L * d * M + 2 * L * M * (dv + 1)) * units,
        "tc_out_kernel": (2 * L * d * M + 2 * L * M * (dv + 1)) * units,
        "tc_featq_kernel": 2 * L * d * M * units,
        "tc_causal_out_kernel": (2 * L * M * (dv + 1) + 2 * L * 128 * M + 2 * L * 128 * dv) * units,
    }
    bytes_of = {"stats_kernel": 2 * L * d * es * units, "tc_stats_kernel": 2 * L * d * es * units, "expshift_kernel": 2 * L * M * 4 * units,
                "rowterm_kernel": L * d * es * units, "groupmax_kernel": L * M * 4 * units,
                "tc_rowterm_kernel": L * d * es * units,
                "tc_causal_prefix_kernel": ((L + 127) // 128) * (65 * M * 2 + 80 * M * 2) * units}
    if name in flops_of and flops_of[name]:
        fl = flops_of[name] * (per_launch if name in ("logits_kernel", "kv_kernel", "out_kernel", "scores_kernel") and
                               k["launches_per_step"] > 1 else 1.0)
        ach = fl / t / 1e12
        return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": ach / peaks["bf16_tflops"], "traffic": NCU_TRAFFIC.get((w.name, name)), "peak_source": peaks["source"]}
    if name == "fit_kernel":
        # fp64 arithmetic of the fit.  Direct solver (d <= 64): Householder tridiagonalisation 4/3 d^3, Sturm counts
        # (one grid of 512 points, then P = 512/d points per eigenvalue and step, 4 flops per recurrence step),
        # reflectors applied back 2 d^3, four d^3 products (orthogonality check, correction, V A, (V A) V^T) 8 d^3;
        # ADERF adds the elimination for L and L^-1 (2 d^3) and six more products (12 d^3).  Jacobi sweeps, when the
        # direct result needs them (always for d = 128): per round and group the 2 x 2 blocks of A (8 multiplies +
        # 8 multiply-adds each) and d/2 * d row-pair entries of V^T (2 multiplies + 2 multiply-adds each).
        # Peak = 64 fp64 FMA per clock and SM.
        h = d // 2
        blocks = h * (h + 1) // 2 if d <= 64 else h * h
        per_group = work.get("fit_sweeps", 0.0) * (d - 1) * (blocks * 24 + h * d * 6)
        if d <= 64 and w.variant in ("sderf", "aderf"):
            lanes = 512 // d
            steps = {8: 13, 16: 10, 32: 8}[lanes]
            per_group += (4.0 / 3.0 + 2.0 + 8.0) * d ** 3 + (512 + steps * lanes * d) * d * 4.0
            if w.variant == "aderf":
                per_group += 14.0 * d ** 3
        flops = per_group * units
        peak = 64 * 2 * peaks.get("sm_count", 148) * peaks.get("sm_max_mhz", 1965.0) * 1e6 / 1e12
        ach = flops / t / 1e12
        return {"kernel": name, "bound": "alu", "achieved": ach, "peak": peak, "unit": "TFLOP/s", "frac": ach / peak,
                "traffic": NCU_TRAFFIC.get((w.name, name)) if w.variant == "sderf" else None, "peak_source": "64 fp64 FMA/clk/SM x SMs x max SM clock",
                "note": f"one block per group ({units} of {peaks.get('sm_count', 148)} SMs busy), "
                        f"direct solver + {work.get('fit_sweeps', 0.0):.1f} Jacobi sweeps per group; bound by instruction issue, "
                        f"shared-memory traffic and barrier latency of one block per matrix"}
    by = bytes_of.get(name, work["bytes"]) * (per_launch if k["launches_per_step"] > 1 else 1.0)
    ach = by / t / 1e9
    return {"kernel": name, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC.get((w.name, name)), "peak_source": peaks["source"]}


if __name__ == "__main__":
    main()
