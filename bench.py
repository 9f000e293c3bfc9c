#!/usr/bin/env python
"""Benchmark of the QESGD hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c3|c5|c2|c1|qstep|variance]
  python bench.py --impl reference ...        (the CPU oracle on the host cores)

A step is one pass of the whole path over one batch of synthetic input: all K
simulated workers encode their epoch delta against the anchor (one
qesgd_encode_batch launch) and the server decodes, averages and applies the K
streams (one qesgd_decode_average_apply launch).  The metric is throughput in
fp32-equivalent GB/s: the fp32 delta bytes the calls stand for (4*d*K for encode
plus 4*d*K for decode-average-apply) divided by the device time of the step.

One JSON line is printed by rank 0.  With N > 1 every rank runs an independent
replica on its own GPU (the path has no exchange step); the time is the maximum
over ranks and the value the sum of the work of all ranks over that time.  Started
plainly with --gpus N (no WORLD_SIZE in the environment) the script starts the N
ranks itself.

The default line (C4) also carries `sustained` (the same step for most of a second,
with the SM clock sampled from its first step: the figure under the power cap),
`cpu_baseline` / `cpu_baseline_all_cores` (the oracle on one thread and on all host
cores) and `configs`: C1, C2 at d = 2^24, C3 and C5 at three bucket sizes in short
form, each with its kernels' times, fractions of peak and a parity verdict.
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
    return 6650.0, "fallback (no MEASURED_PEAKS.json beside bench.py)"


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

    def __init__(self, gpu_index, wait_first=False):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        # nvidia-smi needs a few hundred milliseconds before its first line: a region that
        # wants samples from its very start waits for that line (at most 3 s)
        t0 = time.time()
        while wait_first and self.proc is not None and time.time() - t0 < 3.0:
            if os.path.getsize(self.tmp.name) > 0:
                break
            time.sleep(0.02)

    def stop(self, tail=0.25):
        if self.proc is None:
            return None
        time.sleep(tail)
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
    from paper_1901_03040_b200 import synthetic
    d, K = w["d"], w["K"]
    stride = (d + 7) // 8 * 8
    anchor = synthetic.device_normal_f32((d,), synthetic.ANCHOR_SIGMA, seed + 1, device)
    locs = synthetic.device_normal_f32((K, stride), w["sigma"], seed + 2, device,
                                       outlier_prob=w["outlier"])
    locs[:, :d] += anchor            # local_k = fl32(anchor + z_k)
    return anchor, locs, stride


def round_config(w, world):
    """The `config` object of a round workload; the reference arm prints the same one."""
    d, K = w["d"], w["K"]
    return {"workload": w["name"], "d": d, "K": K, "bits": w["bits"], "s": w["s"], "bucket": w["bucket"],
            "scale_mode": "l2-norm",
            "l2": "inputs (K*d*4 = %.2f GB) larger than L2; the anchor is re-read from L2 by design"
                  % (K * d * 4 / 1e9),
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def clocks_bad(clk):
    if not clk:
        return False
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(clk["reasons"])
    stuck = not clk["reasons"] and clk["sm_mhz"] < 0.6 * clk["sm_max_mhz"]
    return bool(bad) or stuck


class RoundBench:
    """One round workload resident on the device: K locals, the anchor, the parameter, the
    stream buffers.  step() = qesgd_encode_batch + qesgd_decode_average_apply."""

    def __init__(self, w, device, seed=0):
        import torch
        from paper_1901_03040_b200 import qesgd
        self.w, self.device = w, device
        self.stream = torch.cuda.Stream(device)
        self.ctx = qesgd.Context(device.index, self.stream)
        self.anchor, self.locs, self.stride = make_round_inputs(w, device, seed)
        self.param = self.anchor.clone()
        self.codes, self.scales = qesgd.alloc_stream_buffers(w["K"], w["d"], w["bucket"], w["bits"], device)
        torch.cuda.synchronize()

    def encode(self, epoch):
        from paper_1901_03040_b200 import qesgd
        w = self.w
        self.ctx.qesgd_encode_batch(self.locs, self.stride, self.param, w["d"], w["K"], w["bucket"], w["s"],
                                    w["bits"], qesgd.SCALE_NORM, 2024, 0, epoch, self.codes,
                                    self.codes.stride(0), self.scales, self.scales.stride(0))

    def apply(self):
        w = self.w
        self.ctx.qesgd_decode_average_apply(self.param, w["d"], w["K"], self.codes, self.codes.stride(0),
                                            self.scales, self.scales.stride(0), w["bucket"], w["s"], w["bits"])

    def step(self, epoch):
        self.encode(epoch)
        self.apply()

    def timed(self, first_epoch, steps, sampler=None, sampler_tail=0.25, barrier=None):
        """`steps` steps between one event pair, per-kernel events inside.  Returns
        (total ms, encode ms per step, apply ms per step, clocks, launches)."""
        import torch
        launches0 = self.ctx.qesgd_launch_count()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        t_begin = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        t_begin.record(self.stream)
        for i in range(steps):
            ev[i][0].record(self.stream)
            self.encode(first_epoch + i)
            ev[i][1].record(self.stream)
            self.apply()
            ev[i][2].record(self.stream)
        t_end.record(self.stream)
        if barrier is not None:
            barrier()
        else:
            torch.cuda.synchronize()
        clk = sampler.stop(sampler_tail) if sampler else None
        return (t_begin.elapsed_time(t_end), [e[0].elapsed_time(e[1]) for e in ev],
                [e[1].elapsed_time(e[2]) for e in ev], clk, self.ctx.qesgd_launch_count() - launches0)

    def kernel_records(self, enc_ms, daa_ms, peak):
        w = self.w
        d, K = w["d"], w["K"]
        enc_bytes, daa_bytes = round_bytes(w)
        out = {}
        for name, ms, nbytes, elems in (("encode_batch", enc_ms, enc_bytes, d * K),
                                        ("decode_average_apply", daa_ms, daa_bytes, d)):
            avg = statistics.mean(ms)
            gbs = nbytes / (avg * 1e-3) / 1e9
            out[name] = {"avg_ms": avg, "min_ms": min(ms), "algorithmic_bytes": nbytes, "hbm_gbs": gbs,
                         "frac_of_peak": gbs / peak, "frac_of_8000": gbs / 8000.0,
                         "fp32_equiv_gbs": 4.0 * d * K / (avg * 1e-3) / 1e9,
                         "elements_per_s": elems / (avg * 1e-3)}
        return out

    def close(self):
        import torch
        self.ctx.close()
        del self.anchor, self.locs, self.param, self.codes, self.scales
        torch.cuda.empty_cache()


def sampled_bucket_parity(rb, n_buckets, seed=1):
    """One untimed round from param = anchor, then the CPU oracle on `n_buckets` buckets drawn
    over the whole vector (plus the first two, the middle one and the last two): a bucket's
    codes and scale depend only on its own elements and their global indices, so each sampled
    bucket is checked exactly; the applied parameter within 1e-6."""
    import numpy as np
    import torch
    from oracle import qesgd_ref as ref
    from paper_1901_03040_b200 import qesgd
    w = rb.w
    d, K, bits, s, B = w["d"], w["K"], w["bits"], w["s"], w["bucket"]
    rb.param.copy_(rb.anchor)
    torch.cuda.synchronize()          # the copy ran on torch's stream, the library runs on its own
    rb.encode(7)
    rb.apply()
    status = rb.ctx.qesgd_status()
    nb = qesgd.num_buckets(d, B)
    rng = np.random.default_rng(seed)
    picks = sorted(set(rng.integers(0, nb, size=n_buckets).tolist())
                   | {0, min(1, nb - 1), nb // 2, max(0, nb - 2), nb - 1})
    bpb = B * bits // 8
    idx = torch.tensor(picks, device=rb.device)
    g_scales = rb.scales[:, idx].cpu().numpy()
    byte_idx = (idx[:, None] * bpb + torch.arange(bpb, device=rb.device)[None, :]).reshape(-1)
    g_codes = rb.codes[:, byte_idx].cpu().numpy().reshape(K, len(picks), bpb)
    elem_idx = (idx[:, None] * B + torch.arange(B, device=rb.device)[None, :]).reshape(-1).clamp_(max=d - 1)
    h_anchor = rb.anchor[elem_idx].cpu().numpy().reshape(len(picks), B)
    h_param = rb.param[elem_idx].cpu().numpy().reshape(len(picks), B)
    h_locs = rb.locs[:, elem_idx].cpu().numpy().reshape(K, len(picks), B)
    bad = {"codes": 0, "scales": 0, "param": 0}
    for n, j in enumerate(picks):
        lo, hi = j * B, min((j + 1) * B, d)
        m = hi - lo
        r_codes, r_scales = [], []
        for k in range(K):
            c, sc, _ = ref.encode(h_locs[k, n, :m], h_anchor[n, :m], B, s, bits, ref.SCALE_NORM, 2024, k, 7,
                                  i0=lo)
            r_codes.append(c)
            r_scales.append(sc)
            bad["codes"] += int((g_codes[k, n].view(np.uint32) != c).any())
            bad["scales"] += int(g_scales[k, n].view(np.uint32) != sc.view(np.uint32)[0])
        r_scales = np.stack(r_scales)
        want = ref.decode_average_apply(h_anchor[n, :m], np.stack(r_codes), r_scales, B, s, bits)
        tol = 1e-6 * np.maximum(np.abs(want), r_scales.max())
        bad["param"] += int((np.abs(h_param[n, :m].astype(np.float64) - want) > tol).any())
    return {"buckets_checked": len(picks), "workers": K, "codes_bit_exact": bad["codes"] == 0,
            "scales_bit_exact": bad["scales"] == 0, "param_within_1e-6": bad["param"] == 0,
            "status_flags": status}


def sustained_leg(rb, first_epoch, ms_per_step, peak, gpu_index, seconds=0.8):
    """The same step repeated for `seconds`: long enough for the power cap to settle the SM
    clock, with clock samples taken from the first step on.  time x MHz makes runs at different
    clocks comparable (the codec kernels are bound by instruction issue)."""
    steps = int(min(20000, max(50, seconds * 1e3 / max(ms_per_step, 1e-3))))
    sampler = ClockSampler(gpu_index, wait_first=True)
    total_ms, enc_ms, daa_ms, clk, _ = rb.timed(first_epoch, steps, sampler, sampler_tail=0.03)
    rec = {"steps": steps, "seconds": total_ms * 1e-3, "ms_per_step": total_ms / steps,
           "value": 2.0 * 4.0 * rb.w["d"] * rb.w["K"] * steps / (total_ms * 1e-3) / 1e9, "unit": UNIT,
           "kernels": rb.kernel_records(enc_ms, daa_ms, peak), "clocks": clk}
    if clk:
        for name in rec["kernels"]:
            rec["kernels"][name]["ms_x_mhz"] = rec["kernels"][name]["avg_ms"] * clk["sm_mhz"]
    return rec, steps


def run_ours(args):
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
    from paper_1901_03040_b200 import qesgd  # noqa: F401  (raises if the library is missing)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no fallback")
    if local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} wants cuda:{local} but only "
                         f"{torch.cuda.device_count()} device(s) are visible")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if args.workload == "c2":
        line = run_c2(args, device, world, rank)
    elif args.workload == "c1":
        line = run_c1(args, device, world, rank)
    elif args.workload == "qstep":
        line = run_qstep(args, device, world, rank)
    elif args.workload == "variance":
        line = run_variance(args, device, world, rank)
    else:
        line = run_round(args, device, world, rank, local)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_round(args, device, world, rank, local):
    import torch
    import torch.distributed as dist
    w = dict(WORKLOADS[args.workload])
    if args.bucket:
        w["bucket"] = args.bucket
    d, K = w["d"], w["K"]
    rb = RoundBench(w, device)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        rb.step(i)
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    total_ms, enc_ms, daa_ms, clocks, launches = rb.timed(args.warmup, args.steps, sampler, barrier=barrier)
    remeasured = False
    again = 1.0 if (rank == 0 and clocks_bad(clocks)) else 0.0
    _, again = aggregate_over_ranks(0.0, again, world, device, world > 1)
    if again > 0.0:       # thermal or hardware slowdown, or clocks pinned low: measure once more
        remeasured = True
        sampler = ClockSampler(local) if rank == 0 else None
        total_ms, enc_ms, daa_ms, clocks, launches = rb.timed(args.warmup + args.steps, args.steps, sampler,
                                                              barrier=barrier)
    if clocks is not None:
        clocks["remeasured"] = remeasured
        clocks["rejected"] = clocks_bad(clocks)
    status = rb.ctx.qesgd_status()

    fp32_equiv_bytes = 2.0 * 4.0 * d * K * args.steps
    ms_all, units_all = aggregate_over_ranks(total_ms, fp32_equiv_bytes, world, device, world > 1)
    value = units_all / (ms_all * 1e-3) / 1e9
    peak, peak_src = peaks()
    kernels = rb.kernel_records(enc_ms, daa_ms, peak)

    # ---- the same step for most of a second: the figure under the power cap ---------------
    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained:
        sustained, used = sustained_leg(rb, args.warmup + 2 * args.steps, ms_all / args.steps, peak, local,
                                        args.sustained_seconds)

    # ---- end to end: host buffers in, host result out, through the same calls -----------
    e2e = None
    cpu_baseline = cpu_all = parity = None
    if not args.no_e2e:
        stride = rb.stride
        h_locs = torch.empty((K, stride), dtype=torch.float32, pin_memory=True)
        h_locs.copy_(rb.locs)
        h_param = torch.empty((d,), dtype=torch.float32, pin_memory=True)
        torch.cuda.synchronize()
        e2e_steps = max(1, min(args.steps, 3))
        e_begin = torch.cuda.Event(enable_timing=True)
        e_end = torch.cuda.Event(enable_timing=True)
        # The result of a step leaves the device on a second stream while the next step's inputs
        # arrive on the first (the link carries both directions at once); the next step's kernels
        # wait until the parameter they overwrite has been read.
        out_stream = torch.cuda.Stream(device)
        left = None                                  # event: the previous step's result is on the host
        with torch.cuda.stream(rb.stream):
            for i in range(1 + e2e_steps):
                if i == 1:
                    barrier()
                    e_begin.record(rb.stream)
                rb.locs.copy_(h_locs, non_blocking=True)
                if left is not None:
                    rb.stream.wait_event(left)
                rb.step(100000 + i)
                done = torch.cuda.Event()
                done.record(rb.stream)
                with torch.cuda.stream(out_stream):
                    out_stream.wait_event(done)
                    h_param.copy_(rb.param, non_blocking=True)
                    left = torch.cuda.Event()
                    left.record(out_stream)
            rb.stream.wait_event(left)
            e_end.record(rb.stream)
            barrier()
        e2e_ms, e2e_units = aggregate_over_ranks(e_begin.elapsed_time(e_end),
                                                 2.0 * 4.0 * d * K * e2e_steps, world, device,
                                                 world > 1)
        e2e = {"value": e2e_units / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": int(h_locs.numel() * 4), "d2h_bytes_per_step": int(d * 4),
               "steps": e2e_steps,
               "note": "K local vectors copied from pinned host memory, updated parameter copied back "
                       "(on a second stream, beside the next step's inputs)"}
        del h_locs, h_param

    # ---- the CPU oracle on a bounded sample of the same inputs, with a parity check -------
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_baseline, cpu_all, parity = oracle_sample(rb.ctx, w, rb.locs, rb.stride, rb.anchor, device,
                                                      args.cpu_sample_elems)

    traffic = load_traffic("encode", args.workload)
    enc = kernels["encode_batch"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_all / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": round_config(w, world),
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "qesgd_encode_kernel (encode_batch, K workers)",
                     "achieved": enc["hbm_gbs"], "peak": peak, "unit": "GB/s", "frac": enc["frac_of_peak"],
                     "traffic": traffic, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": enc["algorithmic_bytes"], "avg_launch_ms": enc["avg_ms"]},
        "kernels": kernels,
        "status_flags": status,
        "clocks": clocks,
        "sustained": sustained,
        "e2e": e2e,
        "cpu_baseline": cpu_baseline,
        "cpu_baseline_all_cores": cpu_all,
        "parity_on_sample": parity,
    }
    rb.close()
    # ---- the other configurations, each with its kernels' times and a parity verdict ------
    if rank == 0 and world == 1 and args.workload == "c4" and not args.no_configs:
        line["configs"] = other_configs(args, device, peak)
    return line


def other_configs(args, device, peak):
    """C1, C2 (d = 2^24), C3 and C5 (three bucket sizes) in short form: per hot kernel its mean
    time, algorithmic bytes and fraction of the measured and of the nominal 8000 GB/s peak, and
    a parity verdict from the CPU oracle on a sample.  20 timed steps each after 3 warm-ups."""
    import copy
    import torch
    out = {}
    sub = copy.copy(args)
    sub.steps, sub.warmup, sub.d, sub.scale_mode = 20, 3, 0, "norm"
    t0 = time.time()

    def short(kernels):
        keep = ("avg_ms", "min_ms", "algorithmic_bytes", "hbm_gbs", "frac_of_peak", "frac_of_8000")
        return {k: {f: v[f] for f in keep if f in v} for k, v in kernels.items()}

    try:
        c1 = run_c1(sub, device, 1, 0)
        out["c1"] = {"workload": c1["config"]["workload"], "round_ms": c1["value"],
                     "kernels": c1["kernels"], "parity": c1["first_round"].get("oracle"),
                     "loss_before": c1["loss_before"], "loss_after_first_round": c1["loss_after_first_rounds"][0],
                     "clocks": c1.get("clocks")}
    except Exception as exc:  # noqa: BLE001  (one configuration must not take the bench line down)
        out["c1"] = {"error": repr(exc)}
    torch.cuda.empty_cache()
    try:
        sub.steps = 200
        c2 = run_c2(sub, device, 1, 0)
        out["c2"] = {"workload": c2["config"]["workload"], "d": c2["config"]["d"],
                     "launch": c2["config"]["launch"], "kernels": short(c2["kernels"]),
                     "parity": c2["parity_on_sample"], "clocks": c2["clocks"]}
    except Exception as exc:  # noqa: BLE001
        out["c2"] = {"error": repr(exc)}
    torch.cuda.empty_cache()
    sub.steps = 20
    todo = [("c3", dict(WORKLOADS["c3"]), 256)]
    for bucket in (128, 512, 4096):
        w = dict(WORKLOADS["c5"])
        w["bucket"] = bucket
        todo.append((f"c5_bucket{bucket}", w, 256 if bucket < 4096 else 64))
    for name, w, n_buckets in todo:
        try:
            need = w["d"] * (w["K"] * 4.6 + 8.5)
            free, _ = torch.cuda.mem_get_info()
            if free < need * 1.1:
                out[name] = {"skipped": f"needs {need / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free"}
                continue
            rb = RoundBench(w, device, seed=len(name))
            for i in range(3):
                rb.step(i)
            torch.cuda.synchronize()
            sampler = ClockSampler(device.index or 0, wait_first=True)
            _, enc_ms, daa_ms, clk, _ = rb.timed(3, sub.steps, sampler, sampler_tail=0.03)
            rec = {"workload": w["name"], "bucket": w["bucket"],
                   "kernels": short(rb.kernel_records(enc_ms, daa_ms, peak)), "clocks": clk}
            if not args.no_cpu:
                rec["parity"] = sampled_bucket_parity(rb, n_buckets)
            out[name] = rec
            rb.close()
        except Exception as exc:  # noqa: BLE001
            out[name] = {"error": repr(exc)}
        torch.cuda.empty_cache()
    out["seconds"] = time.time() - t0
    return out


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


def oracle_round_on_slices(h_loc, h_anchor, w, epoch, threads):
    """The oracle's round (encode of every worker, then decode-average-apply) on host arrays.
    With threads > 1 the vector is cut into bucket ranges, one per thread: buckets are
    independent, the oracle takes a slice with its global offset, and its C calls release the
    interpreter lock.  Returns (codes [K, words], scales [K, nb], new parameter)."""
    import numpy as np
    from concurrent.futures import ThreadPoolExecutor
    from oracle import qesgd_ref as ref
    K, n = h_loc.shape
    bits, s, B = w["bits"], w["s"], w["bucket"]
    nb = (n + B - 1) // B
    cuts = [min(nb, (nb * t) // threads) for t in range(threads + 1)]
    ranges = [(cuts[t] * B, min(n, cuts[t + 1] * B)) for t in range(threads) if cuts[t + 1] > cuts[t]]

    def work(r):
        lo, hi = r
        cs, ss = [], []
        for k in range(K):
            c, sc, _ = ref.encode(h_loc[k, lo:hi], h_anchor[lo:hi], B, s, bits, ref.SCALE_NORM, 2024, k, epoch,
                                  i0=lo)
            cs.append(c)
            ss.append(sc)
        cs, ss = np.stack(cs), np.stack(ss)
        return cs, ss, ref.decode_average_apply(h_anchor[lo:hi], cs, ss, B, s, bits)

    if len(ranges) == 1:
        parts = [work(ranges[0])]
    else:
        with ThreadPoolExecutor(max_workers=len(ranges)) as pool:
            parts = list(pool.map(work, ranges))
    return (np.concatenate([p[0] for p in parts], axis=1), np.concatenate([p[1] for p in parts], axis=1),
            np.concatenate([p[2] for p in parts]))


def oracle_sample(ctx, w, locs, stride, anchor, device, sample_elems):
    """Time the CPU oracle (as it stands) on the first `sample_elems` elements of every worker,
    once on one thread and once with the bucket ranges spread over all host cores, and compare
    the GPU's output on the same slice with it."""
    import numpy as np
    import torch
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
    r_codes, r_scales, r_param = oracle_round_on_slices(h_loc, h_anchor, w, 7, 1)
    dt = time.perf_counter() - t0
    cores = max(1, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1))
    t0 = time.perf_counter()
    a_codes, a_scales, a_param = oracle_round_on_slices(h_loc, h_anchor, w, 7, cores)
    dt_all = time.perf_counter() - t0
    tol = 1e-6 * np.maximum(np.abs(r_param), np.repeat(r_scales.max(0), B)[:n])
    parity = {"codes_bit_exact": bool((g_codes == r_codes).all()),
              "scales_bit_exact": bool((g_scales.view(np.uint32) == r_scales.view(np.uint32)).all()),
              "param_within_1e-6": bool((np.abs(g_param.astype(np.float64) - r_param) <= tol).all()),
              "all_cores_run_equals_one_core_run": bool((a_codes == r_codes).all() and (a_param == r_param).all()
                                                        and (a_scales == r_scales).all()),
              "elements": int(n), "workers": int(K)}
    what = (f"first {n} elements of each of the {K} workers: encode of every worker, then "
            f"decode-average-apply")
    cpu = {"value": 2.0 * 4.0 * n * K / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{what} ({dt:.1f} s of CPU time)", "seconds": dt,
           "elements_per_s": n * K / dt}
    cpu_all = {"value": 2.0 * 4.0 * n * K / dt_all / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"{what}; bucket ranges spread over {cores} threads ({dt_all:.1f} s)",
               "seconds": dt_all, "elements_per_s": n * K / dt_all}
    return cpu, cpu_all, parity


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
    sampler = ClockSampler(device.index, wait_first=True) if rank == 0 else None
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
    for rec in results.values():
        rec["frac_of_8000"] = rec["hbm_gbs"] / 8000.0
        rec["algorithmic_bytes"] = rec["hbm_gbs"] * 1e9 * rec["avg_ms"] * 1e-3
    if rank == 0 and world == 1 and not args.no_cpu:
        line["parity_on_sample"] = c2_parity(ctx, zs[0], d, B, mode, variants, device)
    else:
        line["parity_on_sample"] = None
    ctx.close()
    return line


def c2_parity(ctx, z, d, B, mode, variants, device, n=1 << 21):
    """Encode and decode of the first n elements (whole buckets) against the CPU oracle, all
    three code widths: codes, scales and decoded values bit for bit."""
    import numpy as np
    import torch
    from oracle import qesgd_ref as ref
    from paper_1901_03040_b200 import qesgd
    n = min(n, d) // B * B
    h = z[:n].cpu().numpy()
    ok = {}
    for bits, s in variants:
        codes, scales = qesgd.alloc_stream_buffers(1, n, B, bits, device)
        out = torch.empty(n, dtype=torch.float32, device=device)
        ctx.qesgd_encode(z, None, n, B, s, bits, mode, 1, 0, 3, codes, scales, fixed_delta=3e-3 / s)
        ctx.qesgd_decode(codes, scales, n, B, s, bits, out)
        torch.cuda.synchronize()
        r_codes, r_scales, _ = ref.encode(h, None, B, s, bits, mode, 1, 0, 3, fixed_delta=3e-3 / s)
        r_out = ref.decode(r_codes, r_scales, n, B, s, bits)
        g_codes = codes.view(-1)[:n * bits // 8].cpu().numpy().view(np.uint32)
        g_scales = scales.view(-1)[:n // B].cpu().numpy()
        ok[f"{bits}bit"] = bool((g_codes == r_codes).all()
                                and (g_scales.view(np.uint32) == r_scales.view(np.uint32)).all()
                                and (out.cpu().numpy().view(np.uint32) == r_out.view(np.uint32)).all())
    return {"elements": int(n), "codes_scales_decoded_bit_exact": ok}


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
    del u, w, zsum, codes, scales
    line["inner_step"] = inner_step_leg(ctx, stream, device, args, mode)
    ctx.close()
    return line


def inner_step_leg(ctx, stream, device, args, mode):
    """Algorithm 2's whole inner iteration on logistic regression, m = 64 rows of d = 2^22 columns
    (a minibatch is 1.07 GB, two of them alternate, so X always comes from HBM): the fused call
    qesgd_lr_qesgd_step (margin pass + one kernel that updates, quantises and writes back) against
    qesgd_lr_sgd_step followed by qesgd_requantize (margin pass, update pass, requantise pass)."""
    import torch
    from paper_1901_03040_b200 import qesgd, synthetic
    m, d, B, s, bits, lr = 64, 1 << 22, 512, 127, 8, 0.1
    X = synthetic.device_normal_f32((2 * m, d), 1.0 / (d ** 0.5), 31, device)
    y = torch.where(synthetic.device_normal_f32((2 * m,), 1.0, 32, device) >= 0, 1.0, -1.0).float()
    w = synthetic.device_normal_f32((d,), synthetic.ANCHOR_SIGMA, 33, device)
    codes, scales = qesgd.alloc_stream_buffers(1, d, B, bits, device)
    out = {"m": m, "d": d, "bits": bits, "bucket": B}
    steps = max(args.steps, 10)
    for name in ("fused", "two_calls"):
        u = w + synthetic.device_normal_f32((d,), 1e-3, 34, device)
        zsum = torch.zeros(d, dtype=torch.float32, device=device)

        def call(i):
            Xb, yb = X[(i % 2) * m:(i % 2 + 1) * m], y[(i % 2) * m:(i % 2 + 1) * m]
            if name == "fused":
                ctx.qesgd_lr_qesgd_step(Xb, yb, m, d, lr, u, w, B, s, bits, mode, 7, 0, i, zsum, codes, scales,
                                        fixed_delta=4e-3 / s)
            else:
                ctx.qesgd_lr_sgd_step(Xb, yb, m, d, lr, u)
                ctx.qesgd_requantize(u, w, d, B, s, bits, mode, 7, 0, i, zsum, codes, scales,
                                     fixed_delta=4e-3 / s)
        for i in range(max(args.warmup, 3)):
            call(i)
        torch.cuda.synchronize()
        n0 = ctx.qesgd_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            call(i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        # X twice (margins, update) + u, anchor, running sum read, u and running sum written + code
        nbytes = 2.0 * m * d * 4 + d * (12.0 + 8.0 + bits / 8.0 + 4.0 / B)
        out[name] = {"ms_per_step": ms, "launches_per_step": (ctx.qesgd_launch_count() - n0) / steps,
                     "algorithmic_bytes": nbytes, "hbm_gbs": nbytes / (ms * 1e-3) / 1e9}
        del u, zsum
    out["fused_over_two_calls"] = out["fused"]["ms_per_step"] / out["two_calls"]["ms_per_step"]
    out["status_flags"] = ctx.qesgd_status()
    return out


def c1_kernel_records(times, n, d, K, B, bits):
    """Mean time of each of the three launches of a C1 round with its algorithmic bytes: every row
    of X once for the local epoch; locals, anchor and streams for the codec calls."""
    per = bits / 8.0 + 4.0 / B
    nbytes = {"local_epoch": float(n) * d * 4, "encode": d * (K * (4 + per) + 4), "apply": d * (K * per + 8)}
    peak = peaks()[0]
    out = {}
    for k, v in times.items():
        ms = statistics.mean(v)
        gbs = nbytes[k] / (ms * 1e-3) / 1e9
        out[k] = {"avg_ms": ms, "min_ms": min(v), "algorithmic_bytes": nbytes[k], "hbm_gbs": gbs,
                  "frac_of_peak": gbs / peak, "frac_of_8000": gbs / 8000.0}
    return out


def run_c1(args, device, world, rank):
    """End-to-end QESGD round on logistic regression: K=4 workers run one local epoch of
    minibatch-64 SGD from the anchor, encode (8-bit, bucket 512), server applies."""
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
        if it == 0:   # the first QESGD round (from w = 0), outside every timed region
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
            "kernels": c1_kernel_records(times, n, d, K, B, bits),
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
                                "sample": "the whole of the first QESGD round: four local epochs, encode of the four "
                                          "workers, decode-average-apply"}
    ctx.close()
    return line


def quantisation_variance(ctx, v, bucket, s, bits, draws, seed=5):
    """Monte-Carlo E||Q(v) - v||^2 of the library's quantiser (encode with anchor = NULL and
    the bucket's L2 norm as scale, then decode) over `draws` epochs of draws, beside Lemma 1's
    closed form sum_i delta_b^2 p_i (1 - p_i), p_i the fractional part of |v_i| / delta_b and
    delta_b = fl32(scale_b / s) the decoder's grid spacing.  v is a device vector; the sums are
    taken in fp64 on the device (measurement only: the path itself is the two library calls)."""
    import torch
    from paper_1901_03040_b200 import qesgd
    d = v.numel()
    codes, scales = qesgd.alloc_stream_buffers(1, d, bucket, bits, v.device)
    out = torch.empty(d, dtype=torch.float32, device=v.device)
    acc = 0.0
    for e in range(draws):
        ctx.qesgd_encode(v, None, d, bucket, s, bits, qesgd.SCALE_NORM, seed, 0, e, codes, scales)
        ctx.qesgd_decode(codes, scales, d, bucket, s, bits, out)
        (ctx.stream or torch.cuda.current_stream()).synchronize()
        acc += float(((out.double() - v.double()) ** 2).sum().item())
    nb = qesgd.num_buckets(d, bucket)
    delta = (scales.view(-1)[:nb] / float(s)).double()              # fl32(scale/s), then exact
    delta_e = delta.repeat_interleave(bucket)[:d]
    r = torch.where(delta_e > 0, v.double().abs() / delta_e.clamp_min(1e-300), torch.zeros_like(delta_e))
    p = r - torch.floor(r)
    closed = float((delta_e ** 2 * p * (1.0 - p)).sum().item())
    bound = float((delta_e ** 2).sum().item()) / 4.0              # d * delta^2 / 4 (proof of Theorem 1)
    return {"monte_carlo": acc / draws, "closed_form": closed, "bound_d_delta2_over_4": bound,
            "norm2": float((v.double() ** 2).sum().item()), "draws": draws}


def run_variance(args, device, world, rank):
    """Gradient compression (the QSGD baseline of Sec. 5: delta = ||g||) against compression of the
    epoch delta (QESGD, Sec. 2.2) on the C1 logistic problem, same code width and bucket: the
    quantisation noise E||Q(v) - v||^2 of a minibatch gradient g and of a local-epoch delta
    z = u - w_t, each against Lemma 1's closed form, and what either scheme adds to the
    parameter per epoch: QSGD quantises every one of the epoch's steps (noise lr^2 * Var per
    step), QESGD quantises once per epoch."""
    import torch
    from paper_1901_03040_b200 import qesgd, synthetic
    n, d, K, batch, lr, B, s, bits = 8192, 65536, 4, 64, 0.1, 512, 127, 8
    if args.d:
        d = args.d
    draws = max(8, min(args.steps, 256))
    stream = torch.cuda.Stream(device)
    ctx = qesgd.Context(device.index, stream)
    X, y, _ = synthetic.logistic_problem(n, d, seed=0)
    tX, ty = torch.from_numpy(X).to(device), torch.from_numpy(y).to(device)
    n_local = n // K
    w = torch.zeros(d, dtype=torch.float32, device=device)
    g = torch.empty(d, dtype=torch.float32, device=device)
    u = torch.zeros((1, d), dtype=torch.float32, device=device)
    torch.cuda.synchronize()
    t0 = time.time()
    ctx.qesgd_lr_gradient(tX[:batch], ty[:batch], batch, d, w, g)
    ctx.qesgd_lr_local_epoch_batch(tX, ty, n_local, d, 1, batch, lr, u, d)
    stream.synchronize()
    z = (u[0] - w).contiguous()
    res = {}
    for bits_, s_ in ((8, 127), (4, 7), (2, 1)):
        rg = quantisation_variance(ctx, g, B, s_, bits_, draws)
        rz = quantisation_variance(ctx, z, B, s_, bits_, draws)
        steps = n_local // batch
        res[f"{bits_}bit"] = {
            "gradient": rg, "epoch_delta": rz,
            "relative_noise": {"gradient": rg["monte_carlo"] / rg["norm2"],
                               "epoch_delta": rz["monte_carlo"] / rz["norm2"]},
            "parameter_noise_per_epoch": {"qsgd_every_step": steps * lr * lr * rg["monte_carlo"],
                                          "qesgd_once": rz["monte_carlo"]},
            "monte_carlo_over_closed_form": {"gradient": rg["monte_carlo"] / rg["closed_form"],
                                             "epoch_delta": rz["monte_carlo"] / rz["closed_form"]}}
    dt = time.time() - t0
    line = {"metric": "quantisation noise E||Q(v)-v||^2, gradient vs epoch delta", "value": dt, "unit": "s",
            "n_gpus": world, "steps": draws, "warmup": 0, "ms_per_step": dt * 1e3 / draws,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": "variance of Q(g) against Q(z) on the C1 logistic problem (worker 0, "
                                   "w = 0, minibatch 64, lr 0.1, bucket 512, L2-norm scale)", "d": d,
                       "draws": draws},
            "gpu_launches": int(ctx.qesgd_launch_count()), "results": res,
            "status_flags": ctx.qesgd_status()}
    ctx.close()
    return line


def c1_first_round(args, rank, world, X, y, u, codes, scales, param, loss, shape):
    """The first QESGD round of C1 looked at from outside the timed region: the loss the unquantised average of
    the workers' parameters would have given (Sec. 5 claims 8 bits lose nothing against plain
    SGD), and, with the CPU oracle, the same round on the host: the oracle's local epochs against
    the GPU's (tolerance), then hand-off parity -- the oracle encodes the GPU's u_k and its codes
    and scales must equal the GPU's bit for bit, its applied parameter within 1e-6."""
    import numpy as np
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
    if rank != 0:          # under torchrun rank 0 alone runs the oracle; the others leave
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
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": round_config(w, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def torchrun_command(gpus, argv, port=None):
    """The command that runs this file as `gpus` ranks on this node, one per GPU."""
    if port is None:
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["c4", "c3", "c5", "c2", "c1", "qstep", "variance"], default="c4")
    ap.add_argument("--bucket", type=int, default=0, help="override the bucket size (c5 sweep)")
    ap.add_argument("--d", type=int, default=0, help="vector length for --workload c2")
    ap.add_argument("--scale-mode", choices=["norm", "max", "fixed"], default="norm",
                    help="bucket scale of --workload c2")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of C1, C2, C3, C5")
    ap.add_argument("--no-sustained", action="store_true")
    ap.add_argument("--sustained-seconds", type=float, default=0.8)
    ap.add_argument("--cpu-sample-elems", type=int, default=25_557_032)
    ap.add_argument("--ref-sample-elems", type=int, default=4_194_304)
    args = ap.parse_args(argv)
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    launched = "WORLD_SIZE" in os.environ
    if launched and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={os.environ['WORLD_SIZE']}: start "
                         f"one rank per GPU (torchrun --nproc-per-node {args.gpus}) or drop the variable")
    if args.impl == "reference":
        run_reference(args)
        return 0
    if args.gpus > 1 and not launched:
        # started plainly with --gpus N: become N ranks, one replica per GPU
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} but {have} CUDA device(s) visible")
        return subprocess.call(torchrun_command(args.gpus, argv))
    run_ours(args)
    return 0


if __name__ == "__main__":
    sys.exit(main())
