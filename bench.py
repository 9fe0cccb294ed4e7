#!/usr/bin/env python
"""Benchmark of the WERSA attention forward on B200: tokens/s at n = 128k and fraction of roofline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one whole forward pass of the operator (all kernels, all heads) on one batch of
synthetic input.  With N > 1 (torchrun) every rank runs the same per-GPU workload on its own
GPU (slabs are independent: no data-path collective, weak scaling); times are CUDA-event times,
max over ranks.  Rank 0 prints ONE JSON line.

--impl reference times the float64 CPU oracle (oracle/) on the host cores instead.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "WERSA attn tokens/sec on 1 B200 at n=128k (device-timed), % of roofline"
DEFAULT_WORKLOAD = "cfg4_long_bf16"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def fp32_alu_tflops(sms, sm_max_mhz):
    """fp32 FFMA peak behind the fp32 kernels: SMs x 128 lanes x 2 flop x maximum SM clock."""
    return sms * 128 * 2 * sm_max_mhz * 1e6 / 1e12


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def load_traffic():
    """DRAM bytes per token-head per forward kernel from the tracked ncu summary, or ({}, reason) when the
    kernel sources have changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "forward_dram_traffic.txt")
    if not os.path.exists(path):
        return {}, "no capture on file"
    fields = {}
    with open(path) as fh:
        for line in fh:
            if line.startswith("#") or ":" not in line:
                continue
            key, val = line.split(":", 1)
            fields[key.strip()] = val.strip()
    h = hashlib.sha256()
    for rel in fields.get("source_files", "").split():
        with open(os.path.join(ROOT, rel), "rb") as fh:
            h.update(fh.read())
    where = f"profiles/forward_dram_traffic.txt (ncu capture at commit {fields.get('captured_at_commit', '?')}, scaled by token-heads)"
    if h.hexdigest() != fields.get("source_sha256"):
        return {}, "stale: kernel sources changed since " + where
    out = {}
    for key, val in fields.items():
        try:
            out[key] = float(val)
        except ValueError:
            pass
    return out, where


def workload_string(cfg):
    return (f"{cfg['name']}: B={cfg['B']} H={cfg['H']} n={cfg['n']} d={cfg['d']} L={cfg['L']} "
            f"m={cfg['m']} {cfg['dtype']}")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, smax, reasons, power = [], [], set(), []
        with open(self.path) as fh:
            for line in fh:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    smax.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


def oracle_sample_rate(cfg, inp, budget_s):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: the first
    `heads` heads and the first `n_s` tokens of each (a multiple of 2^L), sized for ~budget_s.
    Returns (tokens/s in whole-token units i.e. token-heads / H / s, description, threads, seconds)."""
    from oracle import wersa_oracle as orc
    threads = orc.threads()
    H, n, L = cfg["H"], cfg["n"], cfg["L"]
    heads = max(1, min(H, threads))
    per_thread_rate = 2.0e4                 # token-heads / s / thread, order of magnitude at m=256
    n_s = int(min(n, max(2 ** L, budget_s * per_thread_rate * (256.0 / cfg["m"]))))
    n_s = max(2 ** L, (n_s // 2 ** L) * 2 ** L)
    sl = (slice(0, cfg["B"]), slice(0, heads), slice(0, n_s))
    Q, K, V = inp["Q"][sl], inp["K"][sl], inp["V"][sl]
    gw, gb = inp["gate_w"][:heads], inp["gate_b"][:heads]
    t0 = time.perf_counter()
    orc.forward(Q, K, V, inp["W"], float(inp["beta"][0]), gw, gb, inp["omega"], L)
    dt = time.perf_counter() - t0
    token_heads = cfg["B"] * heads * n_s
    used = min(threads, cfg["B"] * heads)
    desc = (f"oracle forward on {cfg['B']}x{heads} of {cfg['B']}x{H} slabs, first {n_s} of {n} tokens "
            f"each ({token_heads} token-heads), one run")
    return token_heads / H / dt, desc, used, dt


def run_reference(args, cfg, inp, rank):
    """--impl reference: the CPU oracle on the host cores, rank 0 only."""
    if rank != 0:
        return
    budget = max(0.5, min(20.0, 150.0 / (args.steps + args.warmup)))
    rates, times = [], []
    desc, used = "", 1
    for i in range(args.warmup + args.steps):
        rate, desc, used, dt = oracle_sample_rate(cfg, inp, budget)
        if i >= args.warmup:
            rates.append(rate)
            times.append(dt)
    value = sum(rates) / len(rates)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": workload_string(cfg)},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": used, "kind": "oracle", "sample": desc,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--simt", action="store_true", help="force the fp32 FFMA kernels")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=10)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    import wersa_inputs as wi
    cfg = dict(wi.CONFIGS[args.workload], name=args.workload)

    if args.impl == "reference":
        if rank == 0:
            _, inp = wi.make_config(args.workload)
            run_reference(args, cfg, inp, rank)
        return 0

    import numpy as np
    import torch

    import paper_2507_08637_b200 as wersa
    from wersa_inputs import device_inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))

    # every rank draws its own batch of the same shape (different seed per rank)
    cfg_r, inp = wi.make_config(args.workload, seed=wi.CONFIGS[args.workload]["seed"] + 1000 * rank)
    dtype = cfg["dtype"]
    flags = wersa.WERSA_FLAG_FORWARD_ONLY | (wersa.WERSA_FLAG_SIMT_ONLY if args.simt else 0)
    ctx = wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], dtype=dtype,
                             grad_dtype="f32", device=local_rank, flags=flags)
    dev = device_inputs(inp, dtype, device=f"cuda:{local_rank}")
    fargs = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = torch.empty_like(dev["Q"])
    stream = torch.cuda.current_stream()
    tensor_cores = ctx.uses_tensor_cores()

    def step():
        wersa.wersa_forward(ctx, *fargs, out=O, stream=stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    if ctx.query_status() != 0:
        raise SystemExit("device reported an expired wait during warm-up")

    # ---- timed region: exactly K steps, device-timed on the launching stream -----------------
    sampler = ClockSampler(local_rank)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    total_ms = e0.elapsed_time(e1)
    launches = ctx.launch_count(0) * args.steps

    # ---- per-kernel durations (second pass of K steps with an event behind every kernel) -----
    ctx.set_step_timing(True)
    per_kernel = {}
    for _ in range(args.steps):
        step()
        for name, ms in ctx.step_times(0):
            per_kernel.setdefault(name, []).append(ms)
    ctx.set_step_timing(False)
    clocks = sampler.stop()

    if dist is not None:
        t = torch.tensor([total_ms], device=f"cuda:{local_rank}", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    tokens_per_step = cfg["B"] * cfg["n"] * world
    value = tokens_per_step / (ms_per_step * 1e-3)

    # ---- end to end: wersa_forward_host with HOST buffers, copies inside the timed region -----
    # Every step copies Q, K, V from page-locked host memory, runs the forward and copies O back, all
    # inside the library call.  Two steps are kept in flight (two contexts, each with its own workspace,
    # staging buffers, result buffer and stream), so that the result copy of one step overlaps the input
    # copies of the next; the serial figure (one step at a time on one stream) is reported beside it.
    host_in = [dev[k].cpu().pin_memory() for k in ("Q", "K", "V")]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = host_in[0].numel() * host_in[0].element_size()

    class Lane:
        def __init__(self, lane_ctx, lane_stream):
            self.ctx, self.stream = lane_ctx, lane_stream
            self.dQ, self.dK, self.dV, self.dO = (torch.empty_like(dev["Q"]) for _ in range(4))
            self.hO = torch.empty_like(host_in[0]).pin_memory()

        def step(self):
            wersa.wersa_forward_host(self.ctx, *host_in, self.dQ, self.dK, self.dV, *fargs[3:], self.dO, self.hO,
                                     stream=self.stream)

    ctx2 = wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], dtype=dtype,
                              grad_dtype="f32", device=local_rank, flags=flags)
    lanes = [Lane(ctx, stream), Lane(ctx2, torch.cuda.Stream(device=local_rank))]

    def timed_e2e(n_lanes):
        for lane in lanes[:n_lanes]:
            lane.step()
        barrier()
        e0.record(stream)
        for lane in lanes[1:n_lanes]:
            lane.stream.wait_event(e0)
        for i in range(args.e2e_steps):
            lanes[i % n_lanes].step()
        for lane in lanes[1:n_lanes]:
            done = torch.cuda.Event()
            done.record(lane.stream)
            stream.wait_event(done)
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device=f"cuda:{local_rank}", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return tokens_per_step / (ms / args.e2e_steps * 1e-3)

    e2e_serial = timed_e2e(1)
    e2e_value = timed_e2e(2)
    if not torch.equal(lanes[0].hO, O.cpu()) or not torch.equal(lanes[1].hO, lanes[0].hO):
        raise SystemExit("end-to-end result differs from the device-resident forward")
    if ctx.query_status() != 0 or ctx2.query_status() != 0:
        raise SystemExit("device reported an expired wait during the end-to-end steps")

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    # ---- roofline of the dominant kernel -----------------------------------------------------
    peaks, peak_kind = load_peaks()
    sms = torch.cuda.get_device_properties(local_rank).multi_processor_count
    sm_max_mhz = float(clocks.get("sm_max_mhz") or peaks.get("sm_max_mhz") or 1965.0)
    # Which bf16 peak is the denominator: the burst figure while the clocks stay at their maximum, the
    # sustained one once the timed region is long enough for the power cap to pull them down.
    sustained = ("sw_power_cap" in clocks.get("reasons", []) and clocks.get("sm_mhz") and clocks.get("sm_max_mhz")
                 and clocks["sm_mhz"] < 0.985 * clocks["sm_max_mhz"] and "bf16_tflops_sustained" in peaks)
    tensor_peak = float(peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"])
    regime = "sustained" if sustained else "burst"
    TH = cfg["B"] * cfg["H"] * cfg["n"]
    d, m = cfg["d"], cfg["m"]
    s_bytes = 2 if dtype == "bf16" else 4
    avg = {k: sum(v) / len(v) for k, v in per_kernel.items()}
    tot = sum(avg.values())
    dom = max(avg, key=avg.get)
    # algorithmic work of each step per launch
    m_launch = min(m, 256)                           # feature maps wider than 256 run one launch per 256 features
    unit_flops = TH * (4 * d * m_launch + 2 * m_launch)   # one projection + one (m x d) contraction per token-head
    flops = {"tc_kside": unit_flops, "tc_qside": unit_flops, "simt_kside": unit_flops, "simt_qside": unit_flops}
    bytes_ = {"qmean_gate": TH * d * s_bytes, "haar_filter_q": TH * d * (s_bytes + 4),
              "haar_filter_k": TH * d * (s_bytes + 4),
              "tc_kside": 2 * TH * d * s_bytes,      # K and V read once
              "tc_qside": 2 * TH * d * s_bytes,      # Q read once, O written once
              # feature groups: G outputs of 64 columns and G denominators in, O out
              "combine_groups": TH * ((m // 256) * (64 * s_bytes + 4) + d * s_bytes)}
    ncu_bytes_per_th, traffic_source = load_traffic()
    if dom in flops:
        if dom.startswith("tc_"):
            bound, peak, unit = "tensor", tensor_peak, "TFLOP/s"
        else:
            bound, peak, unit = "alu", fp32_alu_tflops(sms, sm_max_mhz), "TFLOP/s"
        achieved = flops[dom] / (avg[dom] * 1e-3) / 1e12
    else:
        bound, peak, unit = "hbm", float(peaks["hbm_gbs"]), "GB/s"
        achieved = bytes_.get(dom, 0) / (avg[dom] * 1e-3) / 1e9
    # (the counters were taken with 64-column heads and one feature group: other shapes move other bytes)
    traffic = ncu_bytes_per_th[dom] * TH if (tensor_cores and dtype == "bf16" and dom in ncu_bytes_per_th and d == 64
                                             and m <= 256) else None
    roofline = {"kernel": dom, "bound": bound, "achieved": achieved, "peak": peak, "unit": unit,
                "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_source,
                "peak_source": f"{peak_kind} ({regime})" if bound == "tensor" else
                               (peak_kind if bound == "hbm" else f"derived: {sms} SM x 128 FFMA x 2 x {sm_max_mhz:.0f} MHz"),
                "kernel_ms": avg, "kernel_share": {k: v / tot for k, v in avg.items()},
                "timing": "CUDA events behind every kernel, second pass of K steps"}
    if dom in flops and dom in bytes_:   # the tensor-core kernels sit on the ridge: report the HBM side too
        roofline["hbm_gbs_achieved"] = bytes_[dom] / (avg[dom] * 1e-3) / 1e9
        roofline["hbm_frac"] = roofline["hbm_gbs_achieved"] / float(peaks["hbm_gbs"])
    # whole-path roofline: slower of FLOPs at tensor peak and bytes at HBM bandwidth
    path_flops = TH * (8 * d * m + 4 * m)
    path_bytes = TH * 4 * d * s_bytes
    t_roof = max(path_flops / (tensor_peak * 1e12), path_bytes / (float(peaks["hbm_gbs"]) * 1e9))
    t_nom = max(path_flops / 2.25e15, path_bytes / 8.0e12)
    path = {"roofline_us": t_roof * 1e6, "frac": t_roof / (ms_per_step * 1e-3), "peaks": f"{peak_kind} ({regime})",
            "roofline_us_nominal": t_nom * 1e6, "frac_nominal": t_nom / (ms_per_step * 1e-3),
            "flops": path_flops, "bytes": path_bytes}

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if tensor_cores else "f32",
        "data": "synthetic",
        "config": {"workload": workload_string(cfg), "per_gpu": True,
                   "l2": "inputs+output 4 x %.0f MB per step exceed the 126 MB L2" % (TH * d * s_bytes / 1e6),
                   "kernels": "tcgen05 bf16, fp32 accumulate" if tensor_cores else "fp32 FFMA", "storage": dtype},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": args.e2e_steps, "serial_value": e2e_serial,
                "what": "wersa_forward_host from page-locked host tensors, two steps in flight (the result copy "
                        "of one overlaps the input copies of the next); serial_value = one step at a time"},
        "gpu_launches": launches,
        "roofline": roofline,
        "path_roofline": path,
    }
    if cfg.get("backward"):   # training-shaped workload: also time forward + backward (device events)
        ctx_t = wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], dtype=dtype,
                                   grad_dtype="f32", device=local_rank,
                                   flags=wersa.WERSA_FLAG_SIMT_ONLY if args.simt else 0)
        for _ in range(3):
            wersa.wersa_forward(ctx_t, *fargs, out=O, stream=stream)
            wersa.wersa_backward(ctx_t, *fargs, dev["dO"], stream=stream)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(20):
            wersa.wersa_forward(ctx_t, *fargs, out=O, stream=stream)
            wersa.wersa_backward(ctx_t, *fargs, dev["dO"], stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        tms = e0.elapsed_time(e1) / 20
        line["training_step"] = {"ms_per_step": tms, "tokens_per_s": cfg["B"] * cfg["n"] / (tms * 1e-3),
                                 "what": "forward + backward, device-timed, 20 steps",
                                 "launches": ctx_t.launch_count(0) + ctx_t.launch_count(1)}
    # the stand-alone Haar filter pass X -> T_f(X) on this workload's Q: a pure streaming kernel, read + write
    hf = torch.linspace(0.5, 1.5, cfg["B"] * cfg["H"] * (cfg["L"] + 1), device=f"cuda:{local_rank}",
                        dtype=torch.float32).view(cfg["B"] * cfg["H"], cfg["L"] + 1)
    XF = torch.empty_like(dev["Q"])
    for _ in range(3):
        ctx.haar_filter(dev["Q"], hf, out=XF, stream=stream)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(20):
        ctx.haar_filter(dev["Q"], hf, out=XF, stream=stream)
    e1.record(stream)
    torch.cuda.synchronize()
    hms = e0.elapsed_time(e1) / 20
    hbytes = 2 * dev["Q"].numel() * dev["Q"].element_size()
    line["haar_filter_pass"] = {"ms": hms, "bytes": hbytes, "achieved_gbs": hbytes / (hms * 1e-3) / 1e9,
                                "peak_gbs": float(peaks["hbm_gbs"]),
                                "frac": hbytes / (hms * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                                "what": "wersa_haar_filter on Q (read once, written once), 20 launches, device-timed"}
    del XF
    if not args.no_cpu_baseline:
        rate, desc, used, _ = oracle_sample_rate(cfg, inp, 15.0)
        line["cpu_baseline"] = {"value": rate, "unit": "tokens/s", "cores": used, "kind": "oracle",
                                "sample": desc, "host_cores": os.cpu_count()}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
