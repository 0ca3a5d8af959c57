"""Benchmark of the SMaLL layer set on B200.

python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--math fp32|tf32|3xtf32] [--no-sweep] [--no-overlap]

One step = one pass of the 8-layer residual CNN (batch 256 per GPU) through small_run_net, inputs resident in HBM.
The JSON line also carries the end-to-end figure from host buffers (small_run_net_host), the per-kernel roofline
of the dominant kernel, the GPU-scale layer sweep (GFLOP/s and fraction of each layer's roofline) and the CPU
oracle timed on the host cores.  `--impl reference` times the CPU oracle alone.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from synth import configs

WORKLOAD = "residual_cnn"          # the 8-layer residual CNN, batch 256
METRIC, UNIT = "inferences_per_sec", "inferences/s"
FLUSH_BYTES = 256 << 20            # larger than the 126 MB L2
TOL = {"fp32": 1e-5, "tf32": 2e-3, "3xtf32": 1e-5}

# DRAM traffic per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture of
# this file's network step, averaged over the kernel's launches in one step).  It is reported only while the kernel's
# source still has the hash it had when the counters were taken.
TRAFFIC = {
    "conv_3xtf32_warp_mma": {"bytes_per_launch": 27034410.7, "source": "paper_2303_04769_b200/csrc/conv_mma.cuh",
                             "sha256": "527a631d999499591cd9734e5b054a66bad05b1cbc1ae99376edb6c78c01de45"},
    "conv_tf32_warp_mma": {"bytes_per_launch": 27010986.7, "source": "paper_2303_04769_b200/csrc/conv_mma.cuh",
                           "sha256": "527a631d999499591cd9734e5b054a66bad05b1cbc1ae99376edb6c78c01de45"},
    "conv_3xtf32_tensor": {"bytes_per_launch": 22910037.0, "source": "paper_2303_04769_b200/csrc/conv_tc.cu",
                           "sha256": "46edea15c263baabda86068dc7269c4601c27973edc2dd8509505bfd06924f4c"},
    "conv_tf32_tensor": {"bytes_per_launch": 24391387.0, "source": "paper_2303_04769_b200/csrc/conv_tc.cu",
                         "sha256": "46edea15c263baabda86068dc7269c4601c27973edc2dd8509505bfd06924f4c"},
}


def measured_traffic(kernel):
    import hashlib
    t = TRAFFIC.get(kernel)
    if not t or t["bytes_per_launch"] is None:
        return None
    try:
        h = hashlib.sha256(open(os.path.join(ROOT, t["source"]), "rb").read()).hexdigest()
    except OSError:
        return None
    return t["bytes_per_launch"] if h == t["sha256"] else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    sm_max_mhz=p.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


def mode_peak_tflops(mode, peaks, sm_count=148):
    """Peak of the arithmetic a convolution runs in: TF32 tensor = half the measured BF16 burst (nominal ratio);
    3xTF32 = a third of that; FP32 = SMs x 128 lanes x 2 x max SM clock."""
    if mode == "tf32":
        return peaks["bf16_burst"] * 0.5
    if mode == "3xtf32":
        return peaks["bf16_burst"] * 0.5 / 3.0
    return sm_count * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12


def layer_work(row, N, accumulate=False):
    """Algorithmic FLOPs and bytes of one layer from its logical dimensions (each tensor moved once, 4-byte floats)."""
    C, K, H, W, FH, FW, OH, OW = (row[k] for k in ("C", "K", "H", "W", "FH", "FW", "OH", "OW"))
    if row["op"] == "conv":
        fl = 2.0 * N * OH * OW * K * C * FH * FW
        by = 4.0 * (N * C * H * W + N * K * OH * OW * (2 if accumulate else 1) + K * C * FH * FW + K)
    elif row["op"] == "dwconv":
        fl = 2.0 * N * OH * OW * C * FH * FW
        by = 4.0 * (N * C * (H * W + OH * OW) + C * FH * FW + C)
    elif row["op"] == "pool":
        fl = 1.0 * N * C * OH * OW * FH * FW
        by = 4.0 * N * C * (H * W + OH * OW)
    elif row["op"] == "fc":
        fl = 2.0 * N * C * K
        by = 4.0 * (N * C + N * K + C * K + K)
    else:
        fl, by = 0.0, 8.0 * N * C * H * W
    return fl, by


class ClockSampler:
    """nvidia-smi sampled every 100 ms while the timed region runs (reading only; nothing is set)."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [s.strip() for s in line.split(",")]
            if len(f) < 6:
                continue
            try:
                mhz.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for name, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(mhz)}


def dist_env(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(value, world, device=None):
    """The slowest rank's time: all-reduce MAX over the job (NCCL on GPUs, gloo in the CPU tests)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value, world, device=None):
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_throughput(units_local, ms_local, world, device=None):
    """Units all ranks processed / the slowest rank's time.  Images are independent, so ranks share nothing."""
    units = sum_over_ranks(units_local, world, device)
    ms = max_over_ranks(ms_local, world, device)
    return units / (ms * 1e-3), ms


# ------------------------------------------------------------------------------------------- CPU oracle legs
def time_oracle_net(batch_cap, target_s=12.0, f32acc=False):
    """The oracle as it stands on the host cores: a bounded sample of the workload (at most the full batch per pass,
    whole passes repeated until about target_s seconds of CPU work are done).  f32acc: the convolutions' sums in a
    float accumulator instead of double (the same loops; a second, fairer CPU figure - parity always uses double)."""
    import oracle
    from oracle import nets
    net = configs.NETWORKS[WORKLOAD]()
    params = configs.make_params(net)
    probe = 8
    x = configs.make_input(net, probe)
    t0 = time.perf_counter()
    nets.run_net(net, params, x, f32acc=f32acc)
    dt = time.perf_counter() - t0
    n = int(max(probe, min(batch_cap, probe * target_s / max(dt, 1e-6))))
    x = configs.make_input(net, n)
    passes, total = 0, 0.0
    while passes == 0 or (total < target_s and passes < 64):
        t0 = time.perf_counter()
        nets.run_net(net, params, x, f32acc=f32acc)
        total += time.perf_counter() - t0
        passes += 1
    return n * passes / total, n, total, oracle.num_threads(), passes


def reference_arm(args):
    rank, world, _ = dist_env(args.gpus)
    if rank != 0:
        return
    net = configs.NETWORKS[WORKLOAD]()
    # every step is a bounded sample of the workload, sized so that the whole run stays within a few minutes:
    # set-up and the size of the sample are fixed once, a step is `passes` passes over `n_used` images
    import oracle
    from oracle import nets
    params = configs.make_params(net)
    per_step_s = max(0.02, min(6.0, 100.0 / (args.steps + args.warmup)))
    probe = 8
    x = configs.make_input(net, probe)
    nets.run_net(net, params, x)                            # first call: builds and loads the C oracle
    t0 = time.perf_counter()
    nets.run_net(net, params, x)
    dt = time.perf_counter() - t0
    n_used = int(max(probe, min(net["batch"], probe * per_step_s / max(dt, 1e-6))))
    passes = max(1, int(per_step_s / max(dt * n_used / probe, 1e-6)))
    x = configs.make_input(net, n_used)
    cores = oracle.num_threads()
    rates = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        for _ in range(passes):
            nets.run_net(net, params, x)
        el = time.perf_counter() - t0
        if i >= args.warmup:
            rates.append(n_used * passes / el)
    value = sum(rates) / len(rates)
    ms = 1e3 * net["batch"] / value                     # one full batch at the sampled rate
    sample = (f"{n_used} of {net['batch']} images per pass, {passes} passes per step (about {per_step_s:.2f} s), "
              "double accumulation, OpenMP; ms_per_step is scaled to the full batch")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64 accumulate over f32 data", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: 8-layer residual CNN, 3x32x32 input, batch {net['batch']}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------- GPU legs
def gpu_main(args):
    import torch
    from paper_2303_04769_b200 import binding as B
    from paper_2303_04769_b200 import build as lib_build
    from paper_2303_04769_b200.net import Net

    rank, world, local = dist_env(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        lib_build.build()
    if world > 1:
        dist.barrier()
    ctx = B.small_init(local)
    if args.no_overlap:
        B.small_set_layer_overlap(ctx, False)
    peaks = load_peaks()
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count

    net = configs.NETWORKS[WORKLOAD]()
    N = net["batch"]
    params = configs.make_params(net)
    gnet = Net(ctx, net, params, math=args.math, device=dev)
    c, h, w = gnet.in_shape
    oc, oh, ow = gnet.out_shape
    # rotating input sets, seeded and distinct per rank and slot
    R = 4
    host_in = [torch.from_numpy(configs.make_input(net, N, seed=20230304 + 17 * rank + r)).pin_memory() for r in range(R)]
    in_blk = []
    for r in range(R):
        blk = torch.empty(B.small_packed_elems(N, c, h, w), device=dev)
        B.small_pack(ctx, host_in[r].to(dev), blk, N, c, h, w)
        in_blk.append(blk)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    host_out = torch.empty((N, oc, oh, ow)).pin_memory()
    torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        evs = []
        for i in range(steps):
            flush.zero_()                      # evict L2 between steps
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn(i)
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in evs) / steps

    sampler = ClockSampler(local) if rank == 0 else None
    ms_eager = timed(lambda i: gnet.run(in_blk[i % R]), args.steps, args.warmup)
    # the same call captured once per input set and replayed: the step the headline number times
    step_graphs = []
    for r in range(R):
        gnet.run(in_blk[r])
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            gnet.run(in_blk[r])
        step_graphs.append(g)
    ms_dev = timed(lambda i: step_graphs[i % R].replay(), args.steps, args.warmup)
    def timed_span(fn, steps, warmup):
        """Back-to-back calls, one pair of events around all of them: the end-to-end leg is a pipeline (the library copies
        a call's input while the layers of the call before it run), which per-step brackets would cut apart."""
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    ms_e2e = timed_span(lambda i: gnet.run_host(host_in[i % R], host_out), args.steps, args.warmup)
    clocks = sampler.stop() if sampler else None
    value, ms = whole_job_throughput(N, ms_dev, world, dev)
    e2e_value, _ = whole_job_throughput(N, ms_e2e, world, dev)
    status = B.small_device_status(ctx)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # ---- per-kernel timing of the same network, one launch at a time on the same stream
    def capture(fn, inner=1):
        """CUDA graph of `inner` back-to-back calls of fn (the library only enqueues kernels, so its calls capture)."""
        fn()                                   # once outside the capture: first-use set-up of the kernels
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(inner):
                fn()
        return g

    def time_launch(fn, reps=20, warm=3, inner=1):
        """Device time of one launch: a graph of `inner` back-to-back launches replayed between two events (so that
        host launch overhead does not hide kernels of a few microseconds); minimum and median over `reps`."""
        g = capture(fn, inner)
        for _ in range(warm):
            g.replay()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            e1.synchronize()
            ts.append(e0.elapsed_time(e1) / inner)
        return min(ts), statistics.median(ts)

    gnet.run(in_blk[0])
    layer_table = []
    by_kernel = {}
    for i, (row, L) in enumerate(zip(gnet.layer_rows, net["layers"])):
        # accumulate layers update their destination in place; values drift over repetitions but the work does not
        tmin, tmed = time_launch(lambda i=i: gnet.run_layer(i, in_blk[0]), inner=10)
        fl, by = layer_work(row, N, L.get("accumulate", False))
        kern = row["op"]
        if row["op"] == "conv":
            path = B.small_conv2d_path(ctx, N, row["C"], row["K"], row["H"], row["W"], row["FH"], row["FW"], row["stride"], row["pad"],
                                       B.MATH[args.math])
            kern = f"conv_{args.math}_tensor" if path == 3 else f"conv_{args.math}_warp_mma" if path == 4 else "conv_fp32_cuda_core"
        layer_table.append({"layer": row["name"], "kernel": kern, "us": round(tmed * 1e3, 2), "gflops": round(fl / tmed / 1e6, 1),
                            "gbs": round(by / tmed / 1e6, 1)})
        k = by_kernel.setdefault(kern, {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "launches": 0})
        k["ms"] += tmed; k["flops"] += fl; k["bytes"] += by; k["launches"] += 1
    dom_name, dom = max(by_kernel.items(), key=lambda kv: kv[1]["ms"])
    # the bound of the dominant kernel is the slower of its FLOPs at the peak of its math mode and its bytes at HBM speed
    mode = None
    if dom_name.startswith("conv"):
        mode = "fp32" if dom_name.endswith("cuda_core") else args.math
    t_bytes = dom["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_flops = dom["flops"] / (mode_peak_tflops(mode, peaks, sm_count) * 1e12) if mode else 0.0
    if t_flops > t_bytes:
        peak = mode_peak_tflops(mode, peaks, sm_count)
        ach = dom["flops"] / (dom["ms"] * 1e-3) / 1e12
        roofline = {"bound": "alu" if mode == "fp32" else "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                    "frac": ach / peak, "traffic": measured_traffic(dom_name), "kernel": dom_name, "launches_per_step": dom["launches"],
                    "peak_source": f"{peaks['source']}: " + ("SMs x 128 x 2 x max SM clock" if mode == "fp32" else "BF16 burst x 0.5 (TF32)" + (" / 3" if mode == "3xtf32" else ""))}
    else:
        ach = dom["bytes"] / (dom["ms"] * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                    "traffic": measured_traffic(dom_name), "kernel": dom_name, "launches_per_step": dom["launches"],
                    "peak_source": f"{peaks['source']}: copy bandwidth"}
    if dom_name.endswith("warp_mma"):
        # context: the warp-level MMA this kernel issues runs at 512 TF32 multiply-adds per clock and SM (measured with a
        # stand-alone issue loop), a quarter of the block-level MMA's rate that `peak` above derives from; against that
        # instruction's own roof the kernel's bound is its arithmetic
        wp = sm_count * 512 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12 / (3.0 if args.math == "3xtf32" else 1.0)
        t_w = dom["flops"] / (wp * 1e12)
        roofline["warp_mma_context"] = {"peak_tflops": wp, "frac_of_slower_roof": max(t_w, t_bytes) / (dom["ms"] * 1e-3),
                                        "bound": "tensor (warp-level MMA)" if t_w > t_bytes else "hbm"}
    roofline["algorithmic_flops_per_launch"] = dom["flops"] / dom["launches"]
    roofline["algorithmic_bytes_per_launch"] = dom["bytes"] / dom["launches"]
    roofline["us_per_launch"] = 1e3 * dom["ms"] / dom["launches"]

    # the same step in the other math modes (graph-replayed, fewer steps), for context beside the headline
    other_modes = {}
    if world == 1:
        for m in ("fp32", "tf32", "3xtf32"):
            if m == args.math:
                continue
            onet = Net(ctx, net, params, math=m, device=dev)
            onet.run(in_blk[0])
            torch.cuda.synchronize()
            og = torch.cuda.CUDAGraph()
            with torch.cuda.graph(og):
                onet.run(in_blk[0])
            oms = timed(lambda i: og.replay(), min(args.steps, 200), 5)
            other_modes[m] = {"value": N / (oms * 1e-3), "unit": UNIT, "ms_per_step": oms, "tolerance_rel_l2": TOL[m]}
            del og, onet

    # second workload, for context: the fully-connected autoencoder (batch 4096), each math mode, graph-replayed.  In the
    # tensor-core modes its layers run as 1x1 convolutions over a 1x1 plane on the convolution kernel.
    other_workloads = {}
    if world == 1:
        anet = configs.NETWORKS["autoencoder_fc"]()
        aN = anet["batch"]
        aparams = configs.make_params(anet)
        ax = torch.from_numpy(configs.make_input(anet, aN)).to(dev)
        ablk = torch.empty(B.small_packed_elems(aN, *anet["input"]), device=dev)
        B.small_pack(ctx, ax, ablk, aN, *anet["input"])
        flops = sum(2.0 * aN * L["C"] * L["K"] for L in anet["layers"])
        res = {}
        for m in ("3xtf32", "tf32", "fp32"):
            an = Net(ctx, anet, aparams, math=m, device=dev)
            an.run(ablk)
            torch.cuda.synchronize()
            ag = torch.cuda.CUDAGraph()
            with torch.cuda.graph(ag):
                an.run(ablk)
            ams = timed(lambda i: ag.replay(), min(args.steps, 100), 5)
            res[m] = {"value": aN / (ams * 1e-3), "unit": UNIT, "ms_per_step": ams, "gflops": flops / ams / 1e6}
            del ag, an
        other_workloads["autoencoder_fc"] = {"batch": aN, "layers": len(anet["layers"]), "modes": res}
        del ax, ablk
        # the other two network workloads of the configuration list, at their full batch, same protocol
        for wname in ("dwsep_cnn", "kws_cnn"):
            wnet = configs.NETWORKS[wname]()
            wN = wnet["batch"]
            wparams = configs.make_params(wnet)
            wx = torch.from_numpy(configs.make_input(wnet, wN)).to(dev)
            wblk = torch.empty(B.small_packed_elems(wN, *wnet["input"]), device=dev)
            B.small_pack(ctx, wx, wblk, wN, *wnet["input"])
            res = {}
            for m in ("3xtf32", "tf32", "fp32"):
                wn = Net(ctx, wnet, wparams, math=m, device=dev)
                wn.run(wblk)
                torch.cuda.synchronize()
                wg = torch.cuda.CUDAGraph()
                with torch.cuda.graph(wg):
                    wn.run(wblk)
                wms = timed(lambda i: wg.replay(), min(args.steps, 100), 5)
                res[m] = {"value": wN / (wms * 1e-3), "unit": UNIT, "ms_per_step": wms, "launches": wn.launches()}
                del wg, wn
                if m != "fp32":     # the same network with every depthwise and 1x1 layer launched on its own
                    wn = Net(ctx, wnet, wparams, math=m, device=dev, fuse_dwpw=False)
                    wn.run(wblk)
                    torch.cuda.synchronize()
                    wg = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(wg):
                        wn.run(wblk)
                    wms = timed(lambda i: wg.replay(), min(args.steps, 100), 5)
                    res[m + "_unfused"] = {"value": wN / (wms * 1e-3), "unit": UNIT, "ms_per_step": wms, "launches": wn.launches()}
                    del wg, wn
            other_workloads[wname] = {"batch": wN, "layers": len(wnet["layers"]), "modes": res}
            del wx, wblk

    # the library's own issue-rate probe: what the TF32 pipe sustains with operands resident in shared memory
    probe = None
    if world == 1:
        probe = {}
        for n in (256, 128, 64, 32):
            tf, cpm = B.small_measure_tf32_peak(ctx, n, 4096)
            probe[f"n{n}"] = {"tflops": round(tf, 1), "cycles_per_mma": round(cpm, 1)}

    sweep = None if (args.no_sweep or world > 1) else run_sweep(ctx, B, torch, dev, peaks, sm_count, time_launch, probe["n256"]["tflops"] if probe else None)

    if sweep:
        # the sweep's targets in the retained part of the line: per layer kind and mode the smallest fraction of roofline
        mins, mins_probe = {}, {}
        for r in sweep["rows"]:
            if "frac" not in r or r["layer"].startswith("groupconv") or "fused" in r["layer"]:
                continue
            key = r["layer"] if r["layer"] in ("dw3x3", "maxpool2x2", "relu") else f'{r["layer"]}_{r["mode"]}'
            mins[key] = min(mins.get(key, 9.9), r["frac"])
            if "frac_vs_measured_tf32" in r:
                mins_probe[key] = min(mins_probe.get(key, 9.9), r["frac_vs_measured_tf32"])
        roofline["sweep_min_frac"] = mins
        roofline["sweep_min_frac_vs_measured_tf32"] = mins_probe
    cpu = None
    if world == 1 and not args.no_cpu:
        ips, n_used, dt, cores, passes = time_oracle_net(N)
        cpu = {"value": ips, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"{n_used} of {N} images per pass, {passes} passes, {dt:.1f} s of CPU work, double accumulation, OpenMP"}
        ips32, n32, dt32, _, passes32 = time_oracle_net(N, target_s=6.0, f32acc=True)
        cpu["float_accumulator"] = {"value": ips32, "unit": UNIT,
                                    "sample": f"{n32} of {N} images per pass, {passes32} passes, {dt32:.1f} s of CPU work, the same loops with a float accumulator"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"fp32": "f32", "tf32": "tf32 products, f32 accumulate",
                      "3xtf32": "f32 via 3xTF32 (TF32 part + residual of both operands, f32 accumulate)"}[args.math],
            "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: 8-layer residual CNN, 3x32x32 input, batch {N} per GPU (configs[1])",
                       "math": args.math, "tolerance_rel_l2": TOL[args.math], "l2": "flushed between steps (256 MB write)",
                       "inputs": f"{R} rotating seeded input sets", "parallelism": f"batch shards x{world}, no collective",
                       "launch": "small_run_net captured in a CUDA graph per input set and replayed", "eager_ms_per_step": ms_eager,
                       "layer_overlap": not args.no_overlap},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * N * c * h * w, "d2h_bytes_per_step": 4 * N * oc * oh * ow,
                    "ms_per_step": ms_e2e,
                    "timing": "K back-to-back calls of small_run_net_host between one pair of events (every step copies its input from "
                              "pinned host memory and its result back; the input copy of a step overlaps the layers of the step before "
                              "it); L2 not flushed in this leg: every step's input arrives from the host"},
            "gpu_launches": gnet.launches() * args.steps,
            "clocks": clocks, "roofline": roofline, "other_math_modes": other_modes, "tf32_issue_probe": probe, "other_workloads": other_workloads, "cpu_baseline": cpu, "device_status": status,
            "kernels": {k: {"launches_per_step": v["launches"], "ms": round(v["ms"], 4),
                            "share": round(v["ms"] / sum(x["ms"] for x in by_kernel.values()), 3)} for k, v in by_kernel.items()},
            "layers": layer_table, "sweep": sweep}
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    B.small_shutdown(ctx)


def run_sweep(ctx, B, torch, dev, peaks, sm_count, time_launch, tf32_probe_tflops=None):
    """GPU-scale layer sweep, batch 128: each layer timed alone over rotating buffer sets that together exceed L2;
    GFLOP/s, GB/s and the fraction of the layer's roofline = max(FLOPs / peak of its math mode, bytes / HBM)."""
    import synth
    N = configs.SWEEP_BATCH
    rows = []
    for C, HW in configs.SWEEP_SIZES:
        elems = B.small_packed_elems(N, C, HW, HW)
        sets = max(2, min(48, -(-(1 << 30) // (8 * elems))))         # in + out per set: 1 GiB or more in rotation at every size
        INNER = max(10, sets)                                        # launches per timed graph: every set once or more
        host = synth.uniform((N, C, HW, HW), -1.0, 1.0, 500 + C)
        nchw = torch.from_numpy(host).to(dev)
        ins, outs = [], []
        for s in range(sets):
            blk = torch.empty(elems, device=dev)
            B.small_pack(ctx, nchw, blk, N, C, HW, HW)
            ins.append(blk)
            outs.append(torch.empty(elems, device=dev))
        del nchw
        bias = torch.from_numpy(synth.uniform((C,), -1.0, 1.0, 600 + C)).to(dev)
        state = {"i": 0}

        def rot():
            if state.get("warm"):                # the L2-warm figure: the same buffers in every launch
                return ins[0], outs[0]
            state["i"] = (state["i"] + 1) % sets
            return ins[state["i"]], outs[state["i"]]

        def warm_us(fn, inner=10):
            """The same launch on one fixed buffer set (its tensors may stay in the 126 MB L2): reported apart, labelled."""
            state["warm"] = True
            try:
                return round(time_launch(fn, reps=10, warm=2, inner=inner)[1] * 1e3, 2)
            finally:
                state["warm"] = False

        def record(kind, mode, fl, by, tmin, tmed, bound_mode, us_warm=None):
            t_hbm = by / (peaks["hbm_gbs"] * 1e9)
            t_roof = max(fl / (mode_peak_tflops(bound_mode, peaks, sm_count) * 1e12) if fl and bound_mode else 0.0, t_hbm)
            row = {"layer": kind, "C": C, "HW": HW, "mode": mode, "us_min": round(tmin * 1e3, 2), "us_med": round(tmed * 1e3, 2),
                   "gflops": round(fl / tmed / 1e6, 1), "gbs": round(by / tmed / 1e6, 1),
                   "roofline_us": round(t_roof * 1e6, 2), "frac": round(t_roof / (tmed * 1e-3), 4)}
            if bound_mode in ("tf32", "3xtf32") and tf32_probe_tflops:
                # the same fraction against the library's own measured TF32 issue rate (a third of it for 3xTF32)
                pk = tf32_probe_tflops / (3.0 if bound_mode == "3xtf32" else 1.0)
                row["frac_vs_measured_tf32"] = round(max(fl / (pk * 1e12), t_hbm) / (tmed * 1e-3), 4)
            if us_warm is not None:
                row["us_l2_warm"] = us_warm
            rows.append(row)

        for F, pad, kind in ((3, (1, 1, 1, 1), "conv3x3"), (1, (0, 0, 0, 0), "conv1x1")):
            w = torch.from_numpy(synth.uniform((C, C, F, F), -1.0, 1.0, 700 + C + F)).to(dev)
            wb = torch.empty(B.small_conv_weight_elems(C, C, F, F, B.MATH_3XTF32), device=dev)
            B.small_pack_conv_weights(ctx, w, wb, C, C, F, F, B.MATH_3XTF32)
            fl = 2.0 * N * HW * HW * C * C * F * F
            by = 4.0 * (2 * N * C * HW * HW + C * C * F * F + C)
            for mode in ("fp32", "tf32", "3xtf32"):
                if mode != "fp32" and B.small_conv2d_path(ctx, N, C, C, HW, HW, F, F, 1, pad, B.MATH[mode]) != 3:
                    continue
                def call(mode=mode):
                    a, o = rot()
                    B.small_conv2d(ctx, a, wb, bias, o, N, C, C, HW, HW, F, F, 1, pad, B.RELU | B.MATH[mode])
                slow = mode == "fp32" and F == 3
                tmin, tmed = time_launch(call, reps=5 if slow else 20, warm=2, inner=2 if slow else INNER)
                record(kind, mode, fl, by, tmin, tmed, mode, None if slow else warm_us(call))
            del w, wb
        # group convolution, groups of 32 channels with 32 filters each (G = C / 32): block-diagonal filters on the FP32 kernel,
        # one filter tile per group on the tensor-core kernel
        G = C // 32
        wg = torch.from_numpy(synth.uniform((G, 32, 32, 3, 3), -1.0, 1.0, 900 + C)).to(dev)
        wgb = torch.empty(B.small_group_conv_weight_elems(C, 32, 32, 32, 3, 3), device=dev)
        B.small_pack_group_conv_weights(ctx, wg, wgb, C, 32, 32, 32, 3, 3)

        for mode in ("fp32", "tf32", "3xtf32"):
            def gc(mode=mode):
                a, o = rot()
                B.small_group_conv2d(ctx, a, wgb, bias, o, N, C, 32, 32, 32, HW, HW, 3, 3, 1, (1, 1, 1, 1), B.RELU | B.MATH[mode])
            tmin, tmed = time_launch(gc, reps=10, warm=2, inner=4 if mode == "fp32" else INNER)
            record(f"groupconv3x3_g{G}", mode, 2.0 * N * HW * HW * C * 32 * 9, 4.0 * (2 * N * C * HW * HW + C * 32 * 9 + C), tmin, tmed, mode)
        del wg, wgb
        wdw = torch.from_numpy(synth.uniform((C, 3, 3), -1.0, 1.0, 800 + C)).to(dev)
        wdb = torch.empty(B.small_dw_weight_elems(C, 3, 3), device=dev)
        B.small_pack_dw_weights(ctx, wdw, wdb, C, 3, 3)
        # depthwise 3x3 -> 1x1 as one fused layer (C -> C): no intermediate tensor in the algorithmic bytes
        wpw = torch.from_numpy(synth.uniform((C, C, 1, 1), -1.0, 1.0, 850 + C)).to(dev)
        wpb = torch.empty(B.small_conv_weight_elems(C, C, 1, 1, B.MATH_3XTF32), device=dev)
        B.small_pack_conv_weights(ctx, wpw, wpb, C, C, 1, 1, B.MATH_3XTF32)
        for mode in ("tf32", "3xtf32"):
            if not B.small_dwpw_fused(N, C, C, HW, HW, 1, (1, 1, 1, 1), B.MATH[mode]):
                continue
            def fz(mode=mode):
                a, o = rot()
                B.small_dwpw_conv2d(ctx, a, wdb, bias, wpb, bias, o, None, N, C, C, HW, HW, 1, (1, 1, 1, 1), B.RELU | B.RELU_MID | B.MATH[mode])
            tmin, tmed = time_launch(fz, inner=INNER)
            record("dw3x3+conv1x1_fused", mode, 2.0 * N * HW * HW * C * (9 + C), 4.0 * (2 * N * C * HW * HW + C * C + 12 * C), tmin, tmed, mode)
        del wpw, wpb

        def dw():
            a, o = rot()
            B.small_dwconv2d(ctx, a, wdb, bias, o, N, C, HW, HW, 3, 3, 1, (1, 1, 1, 1), B.RELU)
        tmin, tmed = time_launch(dw, inner=INNER)
        record("dw3x3", "fp32", 2.0 * N * HW * HW * C * 9, 4.0 * (2 * N * C * HW * HW + 10 * C), tmin, tmed, None, warm_us(dw))
        OHW = (HW - 2) // 2 + 1

        def mp():
            a, o = rot()
            B.small_pool2d(ctx, a, o, None, N, C, HW, HW, 2, 2, 2, (0, 0, 0, 0), B.POOL_MAX)
        tmin, tmed = time_launch(mp, inner=INNER)
        record("maxpool2x2", "fp32", 0.0, 4.0 * N * C * (HW * HW + OHW * OHW), tmin, tmed, None, warm_us(mp))

        def rl():
            a, o = rot()
            B.small_relu(ctx, a, o, N, C, HW, HW)
        tmin, tmed = time_launch(rl, inner=INNER)
        record("relu", "fp32", 0.0, 8.0 * N * C * HW * HW, tmin, tmed, None, warm_us(rl))
        # the quantised form of the two convolutions (uint8 tensors, int32 accumulation): operations per second and bytes
        qin = [torch.randint(0, 256, (elems,), dtype=torch.uint8, device=dev) for _ in range(min(sets, 8))]
        qout = [torch.empty(elems, dtype=torch.uint8, device=dev) for _ in range(min(sets, 8))]
        for F, pad, kind in ((3, (1, 1, 1, 1), "qconv3x3"), (1, (0, 0, 0, 0), "qconv1x1")):
            qw = torch.randint(0, 256, (C, C, F, F), dtype=torch.uint8, device=dev)
            qwb = torch.empty(B.small_q_conv_weight_bytes(C, C, F, F), dtype=torch.uint8, device=dev)
            B.small_q_pack_conv_weights(ctx, qw, qwb, C, C, F, F)
            qs = {"i": 0}

            def qc(F=F, pad=pad):
                qs["i"] = (qs["i"] + 1) % len(qin)
                B.small_q_conv2d(ctx, qin[qs["i"]], qwb, None, qout[qs["i"]], N, C, C, HW, HW, F, F, 1, pad, (128, 128, 128, 1 << 20, 40), B.RELU)
            tmin, tmed = time_launch(qc, reps=5, warm=2, inner=4)
            ops, qby = 2.0 * N * HW * HW * C * C * F * F, 1.0 * (2 * N * C * HW * HW + C * C * F * F) + 4.0 * C
            rows.append({"layer": kind, "C": C, "HW": HW, "mode": "uint8", "us_min": round(tmin * 1e3, 2), "us_med": round(tmed * 1e3, 2),
                         "gops": round(ops / tmed / 1e6, 1), "gbs": round(qby / tmed / 1e6, 1)})
            del qw, qwb
        del qin, qout
        del ins, outs
        torch.cuda.empty_cache()
    return {"batch": N, "buffers": "every launch of a timed graph reads and writes its own input/output set, 1 GiB or more in rotation at "
                                   "every size (L2 is 126 MB); us_l2_warm: the same launch on one fixed set, for comparison only",
            "rows": rows}


def single_network(args, ctx, dev, name, batch):
    """One of the small networks, a few graph-replayed steps, for profiler captures of its kernels."""
    import torch
    from paper_2303_04769_b200 import binding as B
    from paper_2303_04769_b200.net import Net
    net = configs.NETWORKS[name]()
    N = batch or net["batch"]
    params = configs.make_params(net)
    x = torch.from_numpy(configs.make_input(net, N)).to(dev)
    blk = torch.empty(B.small_packed_elems(N, *net["input"]), device=dev)
    B.small_pack(ctx, x, blk, N, *net["input"])
    gnet = Net(ctx, net, params, batch=N, math=args.math, device=dev)
    gnet.run(blk)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        gnet.run(blk)
    ts = []
    for i in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        e1.synchronize()
        if i >= args.warmup:
            ts.append(e0.elapsed_time(e1))
    t = statistics.median(ts)
    flops = sum(2.0 * N * L["C"] * L["K"] for L in net["layers"])
    print(json.dumps({"network": name, "batch": N, "math": args.math, "launches": gnet.launches(), "us_med": t * 1e3, "us_min": min(ts) * 1e3,
                      "gflops": flops / t / 1e6, "device_status": B.small_device_status(ctx)}))


def single_layer(args):
    """--layer KIND:C:HW[:BATCH]: one sweep layer, a few launches, for profiler captures (ncu -k ... -c ...)."""
    import torch
    import synth
    from paper_2303_04769_b200 import binding as B
    parts = args.layer.split(":")
    kind, C, HW = parts[0], int(parts[1]), int(parts[2])
    N = int(parts[3]) if len(parts) > 3 else configs.SWEEP_BATCH
    dev = torch.device("cuda", 0)
    ctx = B.small_init(0)
    if kind == "autoencoder":                  # the fully-connected autoencoder as the runner launches it (C, HW ignored)
        return single_network(args, ctx, dev, "autoencoder_fc", N if len(parts) > 3 else None)
    elems = B.small_packed_elems(N, C, HW, HW)
    x = torch.empty(elems, device=dev)
    B.small_pack(ctx, torch.from_numpy(synth.uniform((N, C, HW, HW), -1.0, 1.0, 500 + C)).to(dev), x, N, C, HW, HW)
    y = torch.empty(elems, device=dev)
    bias = torch.from_numpy(synth.uniform((C,), -1.0, 1.0, 600 + C)).to(dev)
    if kind in ("conv3x3", "conv1x1"):
        F, pad = (3, (1, 1, 1, 1)) if kind == "conv3x3" else (1, (0, 0, 0, 0))
        w = torch.from_numpy(synth.uniform((C, C, F, F), -1.0, 1.0, 700 + C + F)).to(dev)
        wb = torch.empty(B.small_conv_weight_elems(C, C, F, F, B.MATH_3XTF32), device=dev)
        B.small_pack_conv_weights(ctx, w, wb, C, C, F, F, B.MATH_3XTF32)
        fn = lambda: B.small_conv2d(ctx, x, wb, bias, y, N, C, C, HW, HW, F, F, 1, pad, B.RELU | B.MATH[args.math])
        fl, by = 2.0 * N * HW * HW * C * C * F * F, 4.0 * (2 * N * C * HW * HW + C * C * F * F + C)
    elif kind == "dw3x3":
        w = torch.from_numpy(synth.uniform((C, 3, 3), -1.0, 1.0, 800 + C)).to(dev)
        wb = torch.empty(B.small_dw_weight_elems(C, 3, 3), device=dev)
        B.small_pack_dw_weights(ctx, w, wb, C, 3, 3)
        fn = lambda: B.small_dwconv2d(ctx, x, wb, bias, y, N, C, HW, HW, 3, 3, 1, (1, 1, 1, 1), B.RELU)
        fl, by = 2.0 * N * HW * HW * C * 9, 4.0 * (2 * N * C * HW * HW + 10 * C)
    elif kind == "maxpool2x2":
        fn = lambda: B.small_pool2d(ctx, x, y, None, N, C, HW, HW, 2, 2, 2, (0, 0, 0, 0), B.POOL_MAX)
        OHW = (HW - 2) // 2 + 1
        fl, by = 0.0, 4.0 * N * C * (HW * HW + OHW * OHW)
    elif kind == "relu":
        fn = lambda: B.small_relu(ctx, x, y, N, C, HW, HW)
        fl, by = 0.0, 8.0 * N * C * HW * HW
    else:
        raise SystemExit(f"unknown layer kind {kind}")
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    fn()                                       # first-use set-up outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()             # one launch, replayed: keeps host launch work out of the timed span
    with torch.cuda.graph(graph):
        fn()
    ts = []
    for i in range(args.warmup + args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        e1.synchronize()
        if i >= args.warmup:
            ts.append(e0.elapsed_time(e1))
    t = statistics.median(ts)
    print(json.dumps({"layer": kind, "C": C, "HW": HW, "batch": N, "math": args.math, "us_med": t * 1e3, "us_min": min(ts) * 1e3,
                      "gflops": fl / t / 1e6, "gbs": by / t / 1e6, "algorithmic_bytes": by, "flops": fl,
                      "device_status": B.small_device_status(ctx)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--math", default="3xtf32", choices=["fp32", "tf32", "3xtf32"],
                    help="arithmetic of the convolutions; the default keeps FP32-level accuracy (1e-5) on the tensor cores")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-overlap", action="store_true",
                    help="launch every layer fully serialised (small_set_layer_overlap off): for profiler captures and comparisons")
    ap.add_argument("--layer", default=None, help="KIND:C:HW[:BATCH] - run one sweep layer only (for profiler captures)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.layer:
        single_layer(args)
    elif args.impl == "reference":
        reference_arm(args)
    else:
        gpu_main(args)


if __name__ == "__main__":
    main()
