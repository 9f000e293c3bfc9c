#!/usr/bin/env python
"""Benchmark of the QESGD hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c3|c5|c2|c1]
  python bench.py --impl reference ...        (the CPU oracle on the host cores)

A step is one pass of the whole path over one batch of synthetic input: all K
simulated workers encode their epoch delta against the anchor (one
qesgd_encode_batch launch) and the server decodes, averages and applies the K
streams (one qesgd_decode_average_apply launch).  The metric is throughput in
fp32-equivalent GB/s: the fp32 delta bytes the calls stand for (4*d*K for encode
plus 4*d*K for decode-average-apply) divided by the device time of the step.

One JSON line is printed by rank 0.  With N > 1 every rank runs an independent
replica on its own GPU (the path has no exchange step); the time is the maximum
over ranks and the value the sum of the work of all ranks over that time.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "encode + decode-average-apply throughput, fp32-equivalent"
UNIT = "GB/s"

WORKLOADS = {
    # ResNet-50-sized flat vector, 16 workers, 2-bit codes: full encode of all workers
    # followed by decode-average-apply, every step.
    "c4": dict(name="C4 full round: K=16 workers, d=25557032 (ResNet-50-sized), 2-bit codes (s=1), "
                    "bucket 256, encode_batch + decode_average_apply per step",
               d=25_557_032, K=16, bits=2, s=1, bucket=256, sigma=1e-4, outlier=0.0),
    "c3": dict(name="C3 server aggregate: K=8 workers, d=11689512 (ResNet-18-sized), 4-bit codes "
                    "(s=7), bucket 512",
               d=11_689_512, K=8, bits=4, s=7, bucket=512, sigma=1e-4, outlier=0.0),
    "c5": dict(name="C5 large sweep: K=8 workers, d=2^30, 4-bit codes (s=7), 1% outliers x100",
               d=1 << 30, K=8, bits=4, s=7, bucket=512, sigma=1e-3, outlier=0.01),
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    return 6650.0, "fallback (earlier measurement on this pool)"


def ideal_comm_speedup(pull_bits, push_bits=32, full_bits=32):
    """Bytes model of the paper's distributed experiment (Sec. 5, last paragraph): a worker
    pushes push_bits per coordinate and pulls pull_bits instead of full_bits each way."""
    return (2.0 * full_bits) / (push_bits + pull_bits)


def round_bytes(w):
    """Compulsory HBM bytes of one launch of each kernel (anchor read once per launch)."""
    d, K, bits, B = w["d"], w["K"], w["bits"], w["bucket"]
    per_stream = bits / 8.0 + 4.0 / B
    enc = d * (K * (4.0 + per_stream) + 4.0)
    daa = d * (K * per_stream + 8.0)
    return enc, daa


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if not sm:
            return None
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm),
                "reasons": sorted(reasons)}


def dist_info():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def aggregate_over_ranks(ms_local, units_local, world, device=None, backend_ready=False):
    """(max time over ranks, sum of units over ranks); identity when world == 1."""
    if world == 1 or not backend_ready:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# --------------------------------------------------------------------- ours ---
def make_round_inputs(w, device, seed=0):
    import torch
    from paper_1901_03040_b200 import synthetic
    d, K = w["d"], w["K"]
    stride = (d + 7) // 8 * 8
    anchor = synthetic.device_normal_f32((d,), synthetic.ANCHOR_SIGMA, seed + 1, device)
    locs = synthetic.device_normal_f32((K, stride), w["sigma"], seed + 2, device,
                                       outlier_prob=w["outlier"])
    locs[:, :d] += anchor            # local_k = fl32(anchor + z_k)
    return anchor, locs, stride


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    world, rank, local = dist_info()
    # build in-tree if the sources are newer (no-op otherwise); there is no fallback path
    from paper_1901_03040_b200 import build as lib_build
    if rank == 0:
        lib_build.build()
    else:           # other ranks wait for rank 0's build instead of racing it
        sources = [os.path.join(lib_build.CSRC, f) for f in os.listdir(lib_build.CSRC)]
        for _ in range(360):
            if os.path.exists(lib_build.LIB) and not lib_build._stale(lib_build.LIB, sources):
                break
            time.sleep(0.5)
    from paper_1901_03040_b200 import qesgd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if args.workload == "c2":
        return run_c2(args, device, world, rank)
    if args.workload == "c1":
        return run_c1(args, device, world, rank)
    if args.workload == "qstep":
        return run_qstep(args, device, world, rank)
    w = dict(WORKLOADS[args.workload])
    if args.bucket:
        w["bucket"] = args.bucket
    d, K, bits, s, B = w["d"], w["K"], w["bits"], w["s"], w["bucket"]

    stream = torch.cuda.Stream(device)
    ctx = qesgd.Context(local, stream)
    anchor, locs, stride = make_round_inputs(w, device)
    param = anchor.clone()
    codes, scales = qesgd.alloc_stream_buffers(K, d, B, bits, device)
    torch.cuda.synchronize()

    def step(epoch):
        ctx.qesgd_encode_batch(locs, stride, param, d, K, B, s, bits, qesgd.SCALE_NORM, 2024, 0,
                               epoch, codes, codes.stride(0), scales, scales.stride(0))
        ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales,
                                       scales.stride(0), B, s, bits)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    def timed_region(first_epoch):
        launches0 = ctx.qesgd_launch_count()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        sampler = ClockSampler(local) if rank == 0 else None
        t_begin = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        t_begin.record(stream)
        for i in range(args.steps):
            ev[i][0].record(stream)
            ctx.qesgd_encode_batch(locs, stride, param, d, K, B, s, bits, qesgd.SCALE_NORM, 2024, 0,
                                   first_epoch + i, codes, codes.stride(0), scales, scales.stride(0))
            ev[i][1].record(stream)
            ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales,
                                           scales.stride(0), B, s, bits)
            ev[i][2].record(stream)
        t_end.record(stream)
        barrier()
        clk = sampler.stop() if sampler else None
        return (t_begin.elapsed_time(t_end), [e[0].elapsed_time(e[1]) for e in ev],
                [e[1].elapsed_time(e[2]) for e in ev], clk, ctx.qesgd_launch_count() - launches0)

    def clocks_bad(clk):
        if not clk:
            return False
        bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clk["reasons"])
        stuck = not clk["reasons"] and clk["sm_mhz"] < 0.6 * clk["sm_max_mhz"]
        return bool(bad) or stuck

    total_ms, enc_ms, daa_ms, clocks, launches = timed_region(args.warmup)
    remeasured = False
    again = 1.0 if (rank == 0 and clocks_bad(clocks)) else 0.0
    _, again = aggregate_over_ranks(0.0, again, world, device, world > 1)
    if again > 0.0:       # thermal or hardware slowdown, or clocks pinned low: measure once more
        remeasured = True
        total_ms, enc_ms, daa_ms, clocks, launches = timed_region(args.warmup + args.steps)
    if clocks is not None:
        clocks["remeasured"] = remeasured
        clocks["rejected"] = clocks_bad(clocks)
    status = ctx.qesgd_status()

    fp32_equiv_bytes = 2.0 * 4.0 * d * K * args.steps
    ms_all, units_all = aggregate_over_ranks(total_ms, fp32_equiv_bytes, world, device, world > 1)
    value = units_all / (ms_all * 1e-3) / 1e9

    # ---- end to end: host buffers in, host result out, through the same calls -----------
    e2e = None
    cpu_baseline = None
    parity = None
    if not args.no_e2e:
        h_locs = torch.empty((K, stride), dtype=torch.float32, pin_memory=True)
        h_locs.copy_(locs)
        h_param = torch.empty((d,), dtype=torch.float32, pin_memory=True)
        torch.cuda.synchronize()
        e2e_steps = max(1, min(args.steps, 3))
        e_begin = torch.cuda.Event(enable_timing=True)
        e_end = torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            for i in range(1 + e2e_steps):
                if i == 1:
                    barrier()
                    e_begin.record(stream)
                locs.copy_(h_locs, non_blocking=True)
                step(1000 + i)
                h_param.copy_(param, non_blocking=True)
            e_end.record(stream)
            barrier()
        e2e_ms, e2e_units = aggregate_over_ranks(e_begin.elapsed_time(e_end),
                                                 2.0 * 4.0 * d * K * e2e_steps, world, device,
                                                 world > 1)
        e2e = {"value": e2e_units / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": int(h_locs.numel() * 4), "d2h_bytes_per_step": int(d * 4),
               "steps": e2e_steps,
               "note": "K local vectors copied from pinned host memory, updated parameter copied back"}
        del h_locs, h_param

    # ---- the CPU oracle on a bounded sample of the same inputs, with a parity check -------
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline, parity = oracle_sample(ctx, w, locs, stride, anchor, device,
                                             args.cpu_sample_elems)

    peak, peak_src = peaks()
    enc_bytes, daa_bytes = round_bytes(w)
    enc_avg = statistics.mean(enc_ms)
    daa_avg = statistics.mean(daa_ms)
    enc_gbs = enc_bytes / (enc_avg * 1e-3) / 1e9
    daa_gbs = daa_bytes / (daa_avg * 1e-3) / 1e9
    traffic = load_traffic("encode", args.workload)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_all / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w["name"], "d": d, "K": K, "bits": bits, "s": s, "bucket": B,
                   "scale_mode": "l2-norm", "l2": "inputs (K*d*4 = %.2f GB) larger than L2; the "
                   "anchor is re-read from L2 by design" % (K * d * 4 / 1e9),
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "qesgd_encode_kernel (encode_batch, K workers)",
                     "achieved": enc_gbs, "peak": peak, "unit": "GB/s", "frac": enc_gbs / peak,
                     "traffic": traffic, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": enc_bytes, "avg_launch_ms": enc_avg},
        "kernels": {
            "encode_batch": {"avg_ms": enc_avg, "min_ms": min(enc_ms), "hbm_gbs": enc_gbs,
                             "frac_of_peak": enc_gbs / peak, "frac_of_8000": enc_gbs / 8000.0,
                             "fp32_equiv_gbs": 4.0 * d * K / (enc_avg * 1e-3) / 1e9,
                             "elements_per_s": d * K / (enc_avg * 1e-3)},
            "decode_average_apply": {"avg_ms": daa_avg, "min_ms": min(daa_ms), "hbm_gbs": daa_gbs,
                                     "frac_of_peak": daa_gbs / peak, "frac_of_8000": daa_gbs / 8000.0,
                                     "fp32_equiv_gbs": 4.0 * d * K / (daa_avg * 1e-3) / 1e9,
                                     "elements_per_s": d / (daa_avg * 1e-3)}},
        "status_flags": status,
        "clocks": clocks,
        "e2e": e2e,
        "cpu_baseline": cpu_baseline,
        "parity_on_sample": parity,
    }
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def load_traffic(kernel, workload):
    """DRAM bytes (read + write) per launch from the committed ncu summary; None when there is
    no capture for this kernel and workload, or the kernel source has changed since."""
    import hashlib
    if kernel == "local_epoch":
        path = os.path.join(ROOT, "profiles", "dram_traffic_bench_c1.txt")
        src = os.path.join(ROOT, "paper_1901_03040_b200", "csrc", "qesgd_lr_epoch.cu")
    else:
        path = os.path.join(ROOT, "profiles", "dram_traffic_bench_c4.txt")
        src = os.path.join(ROOT, "paper_1901_03040_b200", "csrc", "qesgd_codec.cu")
    try:
        with open(src, "rb") as fh:
            sha = hashlib.sha256(fh.read()).hexdigest()
        value, sha_ok = None, False
        with open(path) as fh:
            for line in fh:
                f = line.split()
                if len(f) >= 2 and f[0] == "source_sha256":
                    sha_ok = f[1] == sha
                elif f and f[0] == f"{kernel}:{workload}" and "total_bytes" in f:
                    value = float(f[f.index("total_bytes") + 1])
        return value if sha_ok else None
    except OSError:
        return None


def oracle_sample(ctx, w, locs, stride, anchor, device, sample_elems):
    """Time the CPU oracle (as it stands, one thread) on the first `sample_elems` elements of
    every worker and compare the GPU's output on the same slice with it."""
    import numpy as np
    import torch
    from oracle import qesgd_ref as ref
    from paper_1901_03040_b200 import qesgd
    d, K, bits, s, B = w["d"], w["K"], w["bits"], w["s"], w["bucket"]
    n = min(d, sample_elems) // B * B          # whole buckets only
    nb = n // B
    param = anchor.clone()
    codes, scales = qesgd.alloc_stream_buffers(K, d, B, bits, device)
    ctx.qesgd_encode_batch(locs, stride, param, d, K, B, s, bits, qesgd.SCALE_NORM, 2024, 0, 7,
                           codes, codes.stride(0), scales, scales.stride(0))
    ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales, scales.stride(0),
                                   B, s, bits)
    torch.cuda.synchronize()
    h_loc = locs[:, :n].cpu().numpy()
    h_anchor = anchor[:n].cpu().numpy()
    g_codes = codes[:, :n * bits // 8].cpu().numpy().view(np.uint32)
    g_scales = scales[:, :nb].cpu().numpy()
    g_param = param[:n].cpu().numpy()
    t0 = time.perf_counter()
    r_codes, r_scales = [], []
    for k in range(K):
        c, sc, _ = ref.encode(h_loc[k], h_anchor, B, s, bits, ref.SCALE_NORM, 2024, k, 7)
        r_codes.append(c)
        r_scales.append(sc)
    r_codes, r_scales = np.stack(r_codes), np.stack(r_scales)
    r_param = ref.decode_average_apply(h_anchor, r_codes, r_scales, B, s, bits)
    dt = time.perf_counter() - t0
    tol = 1e-6 * np.maximum(np.abs(r_param), np.repeat(r_scales.max(0), B)[:n])
    parity = {"codes_bit_exact": bool((g_codes == r_codes).all()),
              "scales_bit_exact": bool((g_scales.view(np.uint32) == r_scales.view(np.uint32)).all()),
              "param_within_1e-6": bool((np.abs(g_param.astype(np.float64) - r_param) <= tol).all()),
              "elements": int(n), "workers": int(K)}
    cpu = {"value": 2.0 * 4.0 * n * K / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"first {n} elements of each of the {K} workers: encode of every worker, then "
                     f"decode-average-apply ({dt:.1f} s of CPU time)",
           "seconds": dt}
    return cpu, parity


# --------------------------------------------------- other workloads (own arm) ---
def run_c2(args, device, world, rank):
    """Quantizer microbench: one fp32 delta vector d=2^24, bucket 512, s in {1,7,127}:
    encode, then decode.  Four input sets are rotated so that no launch finds its
    input in L2."""
    import torch
    from paper_1901_03040_b200 import qesgd, synthetic
    d, B = (args.d or (1 << 24)), 512
    R = max(4, (256 << 20) // (4 * d) + 1)      # input sets: together larger than L2
    mode = {"norm": qesgd.SCALE_NORM, "max": qesgd.SCALE_MAX, "fixed": qesgd.SCALE_FIXED}[args.scale_mode]
    stream = torch.cuda.Stream(device)
    ctx = qesgd.Context(device.index, stream)
    zs = [synthetic.device_normal_f32((d,), 1e-3, 10 + r, device) for r in range(R)]
    outs = [torch.empty(d, dtype=torch.float32, device=device) for _ in range(R)]
    variants = [(2, 1), (4, 7), (8, 127)]
    bufs = {bits: [qesgd.alloc_stream_buffers(1, d, B, bits, device) for _ in range(R)]
            for bits, _ in variants}
    peak, peak_src = peaks()
    results = {}
    t_total = 0.0
    graph_launches = 0      # kernel nodes replayed inside the timed regions
    sampler = ClockSampler(device.index) if rank == 0 else None
    for bits, s in variants:
        for kind in ("encode", "decode"):
            def call(i):
                codes, scales = bufs[bits][i % R]
                if kind == "encode":
                    ctx.qesgd_encode(zs[i % R], None, d, B, s, bits, mode, 1, 0, i, codes, scales,
                                     fixed_delta=3e-3 / s)
                else:
                    ctx.qesgd_decode(codes, scales, d, B, s, bits, outs[i % R])
            for i in range(max(args.warmup, R)):
                call(i)
            torch.cuda.synchronize()
            # A launch lasts about as long as one call from Python takes, so the launches are
            # recorded once into CUDA graphs (one rotation over the input sets, plus the
            # remainder) and replayed: exactly `steps` launches between one event pair,
            # back to back on one stream, per-launch time = total / steps.
            full, rest = divmod(args.steps, R)
            graphs = []
            for count in (R, rest):
                if count == 0 or (count == R and full == 0):
                    graphs.append(None)
                    continue
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for i in range(count):
                        call(i)
                graphs.append(g)
            with torch.cuda.stream(stream):
                for g in graphs:            # untimed replay: graph upload and first-run costs
                    if g is not None:
                        g.replay()
                torch.cuda.synchronize()
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(full):
                    graphs[0].replay()
                if graphs[1] is not None:
                    graphs[1].replay()
                e1.record(stream)
            torch.cuda.synchronize()
            graph_launches += args.steps
            avg = e0.elapsed_time(e1) / args.steps
            ms = [avg]
            t_total += avg * args.steps
            nbytes = d * (4.0 + bits / 8.0 + 4.0 / B)
            results[f"{kind}_{bits}bit"] = {
                "avg_ms": avg, "min_ms": min(ms), "hbm_gbs": nbytes / (avg * 1e-3) / 1e9,
                "frac_of_peak": nbytes / (avg * 1e-3) / 1e9 / peak,
                "fp32_equiv_gbs": 4.0 * d / (avg * 1e-3) / 1e9, "elements_per_s": d / (avg * 1e-3)}
    clocks = sampler.stop() if sampler else None
    enc = results["encode_4bit"]
    fp32_bytes = 4.0 * d * 6 * args.steps
    line = {"metric": METRIC, "value": fp32_bytes / (t_total * 1e-3) / 1e9, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": t_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "C2 quantizer microbench: delta ~N(0,1e-3^2), bucket 512, "
                                   "s in {1,7,127}: encode then decode; rotating input sets larger "
                                   "than L2 together", "d": d, "input_sets": R,
                       "scale_mode": args.scale_mode,
                       "launch": "library calls recorded into CUDA graphs and replayed"},
            "gpu_launches": graph_launches,
            "roofline": {"bound": "hbm", "kernel": "qesgd_encode_kernel (4-bit, no anchor)",
                         "achieved": enc["hbm_gbs"], "peak": peak, "unit": "GB/s",
                         "frac": enc["frac_of_peak"], "traffic": load_traffic("encode", "c2"),
                         "peak_source": peak_src},
            "kernels": results, "clocks": clocks}
    if rank == 0:
        print(json.dumps(line))


def run_qstep(args, device, world, rank):
    """Per-step QESGD (Algorithm 2): qesgd_requantize on one vector, d = 2^26 by default, 8-bit
    codes with a caller-given grid spacing (the paper's own choice of delta), bucket 512, running
    sum on.  Algorithmic bytes per element: u, anchor, zsum read (12) + u, zsum written (8) + code
    (1) + scale (4/512)."""
    import torch
    from paper_1901_03040_b200 import qesgd, synthetic
    d, B, s, bits = (args.d or (1 << 26)), 512, 127, 8
    stream = torch.cuda.Stream(device)
    ctx = qesgd.Context(device.index, stream)
    w = synthetic.device_normal_f32((d,), synthetic.ANCHOR_SIGMA, 1, device)
    u = w + synthetic.device_normal_f32((d,), 1e-3, 2, device)
    zsum = torch.zeros(d, dtype=torch.float32, device=device)
    codes, scales = qesgd.alloc_stream_buffers(1, d, B, bits, device)
    mode = {"norm": qesgd.SCALE_NORM, "max": qesgd.SCALE_MAX, "fixed": qesgd.SCALE_FIXED}[args.scale_mode]

    def call(i):
        ctx.qesgd_requantize(u, w, d, B, s, bits, mode, 7, 0, i, zsum, codes, scales,
                             fixed_delta=4e-3 / s)
    for i in range(args.warmup):
        call(i)
    torch.cuda.synchronize()
    launches0 = ctx.qesgd_launch_count()
    sampler = ClockSampler(device.index) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        call(args.warmup + i)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    ms = e0.elapsed_time(e1) / args.steps
    nbytes = d * (12.0 + 8.0 + bits / 8.0 + 4.0 / B)
    peak, peak_src = peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    line = {"metric": "requantize throughput, fp32-equivalent", "value": 4.0 * d / (ms * 1e-3) / 1e9,
            "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "per-step QESGD: qesgd_requantize, 8-bit, bucket 512, running sum",
                       "d": d, "scale_mode": args.scale_mode, "l2": "five streams of 4*d bytes, larger than L2"},
            "gpu_launches": int(ctx.qesgd_launch_count() - launches0),
            "roofline": {"bound": "hbm", "kernel": "qesgd_encode_kernel (requantize)", "achieved": gbs,
                         "peak": peak, "unit": "GB/s", "frac": gbs / peak, "traffic": None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": nbytes},
            "status_flags": ctx.qesgd_status(), "clocks": clocks}
    if rank == 0:
        print(json.dumps(line))


def run_c1(args, device, world, rank):
    """End-to-end QESGD round on logistic regression: K=4 workers run one local epoch of
    minibatch-64 SGD from the anchor, encode (8-bit, bucket 512), server applies."""
    import numpy as np
    import torch
    from paper_1901_03040_b200 import qesgd, synthetic
    n, d, K, batch, lr, B, s, bits = 8192, 65536, 4, 64, 0.1, 512, 127, 8
    stream = torch.cuda.Stream(device)
    ctx = qesgd.Context(device.index, stream)
    X, y, _ = synthetic.logistic_problem(n, d, seed=0)
    tX, ty = torch.from_numpy(X).to(device), torch.from_numpy(y).to(device)
    param = torch.zeros(d, dtype=torch.float32, device=device)
    u = torch.zeros((K, d), dtype=torch.float32, device=device)
    codes, scales = qesgd.alloc_stream_buffers(K, d, B, bits, device)
    n_local = n // K

    def loss(wvec):
        t = -(ty.double() * (tX.double() @ wvec.double()))
        return float(torch.logaddexp(torch.zeros_like(t), t).mean().item())

    loss0 = loss(param)
    times = {"local_epoch": [], "encode": [], "apply": []}
    launches0 = None
    losses = []
    first_round = {}
    for it in range(args.warmup + args.steps):
        if it == args.warmup:
            launches0 = ctx.qesgd_launch_count()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        u.copy_(param.expand(K, d))
        torch.cuda.synchronize()
        e[0].record(stream)
        ctx.qesgd_lr_local_epoch_batch(tX, ty, n_local, d, K, batch, lr, u, d)
        e[1].record(stream)
        ctx.qesgd_encode_batch(u, d, param, d, K, B, s, bits, qesgd.SCALE_NORM, 0, 0, it, codes,
                               codes.stride(0), scales, scales.stride(0))
        e[2].record(stream)
        ctx.qesgd_decode_average_apply(param, d, K, codes, codes.stride(0), scales,
                                       scales.stride(0), B, s, bits)
        e[3].record(stream)
        torch.cuda.synchronize()
        losses.append(loss(param))
        if it == 0:   # round 1 (from w = 0), outside every timed region
            first_round = c1_first_round(args, rank, world, X, y, u, codes, scales, param, loss,
                                         (n_local, d, K, batch, lr, B, s, bits))
        if it >= args.warmup:
            times["local_epoch"].append(e[0].elapsed_time(e[1]))
            times["encode"].append(e[1].elapsed_time(e[2]))
            times["apply"].append(e[2].elapsed_time(e[3]))
    total = sum(sum(v) for v in times.values())
    line = {"metric": "end-to-end QESGD round time", "value": total / args.steps, "unit": "ms",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total / args.steps, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "C1 end-to-end: logistic regression n=8192, d=65536, K=4 workers, "
                                   "one local epoch of minibatch-64 SGD (lr 0.1), 8-bit codes, bucket 512"},
            "gpu_launches": int(ctx.qesgd_launch_count() - launches0),
            "kernels": {k: {"avg_ms": statistics.mean(v)} for k, v in times.items()},
            "roofline": {"bound": "hbm", "kernel": "qesgd_lr_epoch_kernel (local epoch of all workers)",
                         "achieved": n * d * 4 / (statistics.mean(times["local_epoch"]) * 1e-3) / 1e9,
                         "peak": peaks()[0], "unit": "GB/s",
                         "frac": n * d * 4 / (statistics.mean(times["local_epoch"]) * 1e-3) / 1e9 / peaks()[0],
                         "traffic": load_traffic("local_epoch", "c1"), "peak_source": peaks()[1],
                         "algorithmic_bytes_per_launch": float(n * d * 4)},
            "status_flags": ctx.qesgd_status(),
            "x_bytes_per_epoch": int(n * d * 4),
            # algorithmic bytes of the epoch: every row of X once (the minibatch stays on chip
            # between the margin pass and the update pass)
            "local_epoch_gbs": n * d * 4 / (statistics.mean(times["local_epoch"]) * 1e-3) / 1e9,
            "loss_before": loss0, "loss_after_first_rounds": losses[:3], "loss_after_last_round": losses[-1],
            "rounds": len(losses), "first_round": first_round}
    if "oracle" in first_round:
        o = first_round["oracle"]
        line["cpu_baseline"] = {"value": 1e3 * (o["oracle_local_epoch_s"] + o["oracle_codec_s"]), "unit": "ms",
                                "cores": 1, "kind": "oracle",
                                "sample": "the whole of round 1: four local epochs, encode of the four "
                                          "workers, decode-average-apply"}
    if rank == 0:
        print(json.dumps(line))


def c1_first_round(args, rank, world, X, y, u, codes, scales, param, loss, shape):
    """Round 1 of C1 looked at from outside the timed region: the loss the unquantised average of
    the workers' parameters would have given (Sec. 5 claims 8 bits lose nothing against plain
    SGD), and, with the CPU oracle, the same round on the host: the oracle's local epochs against
    the GPU's (tolerance), then hand-off parity -- the oracle encodes the GPU's u_k and its codes
    and scales must equal the GPU's bit for bit, its applied parameter within 1e-6."""
    import numpy as np
    import torch
    n_local, d, K, batch, lr, B, s, bits = shape
    out = {"loss_unquantised_average": loss(u.mean(0)), "loss_quantised": loss(param)}
    if not (rank == 0 and world == 1 and not args.no_cpu):
        return out
    from oracle import qesgd_ref as ref
    h_u = u.cpu().numpy()
    t0 = time.perf_counter()
    w0 = np.zeros(d, dtype=np.float32)
    r_u = np.stack([ref.lr_local_epoch(X[k * n_local:(k + 1) * n_local], y[k * n_local:(k + 1) * n_local],
                                       batch, lr, w0) for k in range(K)])
    t_epoch = time.perf_counter() - t0
    err = np.linalg.norm(h_u.astype(np.float64) - r_u, axis=1) / np.linalg.norm(r_u, axis=1)
    t0 = time.perf_counter()
    enc = [ref.encode(h_u[k], w0, B, s, bits, ref.SCALE_NORM, 0, k, 0) for k in range(K)]
    r_codes, r_scales = np.stack([e[0] for e in enc]), np.stack([e[1] for e in enc])
    r_param = ref.decode_average_apply(w0, r_codes, r_scales, B, s, bits)
    t_codec = time.perf_counter() - t0
    g_codes = codes.cpu().numpy().view(np.uint32).reshape(K, -1)[:, :r_codes.shape[1]]
    g_scales = scales.cpu().numpy()[:, :r_scales.shape[1]]
    g_param = param.cpu().numpy()
    tol = 1e-6 * np.maximum(np.abs(r_param), np.repeat(r_scales.max(0), B)[:d])
    out["oracle"] = {"local_epoch_rel_l2_err_max": float(err.max()), "local_epoch_within_1e-5": bool(err.max() <= 1e-5),
                     "codes_bit_exact": bool((g_codes == r_codes).all()),
                     "scales_bit_exact": bool((g_scales.view(np.uint32) == r_scales.view(np.uint32)).all()),
                     "param_within_1e-6": bool((np.abs(g_param.astype(np.float64) - r_param) <= tol).all()),
                     "oracle_local_epoch_s": t_epoch, "oracle_codec_s": t_codec, "cores": 1}
    return out


# ---------------------------------------------------------------- reference ---
def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step runs the whole path on a
    bounded sample of the workload (first elements of every worker)."""
    world, rank, _ = dist_info()
    if rank != 0:
        return
    import numpy as np
    from oracle import qesgd_ref as ref
    from paper_1901_03040_b200 import synthetic
    w = dict(WORKLOADS[args.workload if args.workload in WORKLOADS else "c4"])
    if args.bucket:
        w["bucket"] = args.bucket
    d, K, bits, s, B = w["d"], w["K"], w["bits"], w["s"], w["bucket"]
    # the sample shrinks with the number of steps so that the whole run takes about a minute
    # (the oracle encodes roughly 3e7 elements per second on one core)
    budget = int(1.4e9 / (K * (args.steps + args.warmup)))
    n = max(8 * B, min(d, args.ref_sample_elems, budget) // B * B)
    anchor = synthetic.anchor_vector(n, seed=1)
    locs = synthetic.worker_locals(anchor, K, w["sigma"], seed=2, outlier_prob=w["outlier"])
    param = anchor.copy()

    def step(epoch):
        nonlocal param
        cs, ss = [], []
        for k in range(K):
            c, sc, _ = ref.encode(locs[k], param, B, s, bits, ref.SCALE_NORM, 2024, k, epoch)
            cs.append(c)
            ss.append(sc)
        param = ref.decode_average_apply(param, np.stack(cs), np.stack(ss), B, s, bits)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    dt = time.perf_counter() - t0
    value = 2.0 * 4.0 * n * K * args.steps / dt / 1e9
    sample = f"first {n} elements of each of the {K} workers per step (one thread)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3 / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64/f32",
            "data": "synthetic",
            "config": {"workload": w["name"], "d": d, "K": K, "bits": bits, "s": s, "bucket": B,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["c4", "c3", "c5", "c2", "c1", "qstep"], default="c4")
    ap.add_argument("--bucket", type=int, default=0, help="override the bucket size (c5 sweep)")
    ap.add_argument("--d", type=int, default=0, help="vector length for --workload c2")
    ap.add_argument("--scale-mode", choices=["norm", "max", "fixed"], default="norm",
                    help="bucket scale of --workload c2")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-sample-elems", type=int, default=25_557_032)
    ap.add_argument("--ref-sample-elems", type=int, default=4_194_304)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
