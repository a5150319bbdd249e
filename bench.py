#!/usr/bin/env python
"""Benchmark of the 4-bit weight-only decode path on the Llama-2-7B linear shapes (decode batch 1).

One step = one pass over the 224 linears of the 32 decoder layers (q, k, v, o, gate, up, down),
i.e. the linears behind one action token; ~3.44 GB of packed weights are streamed per step, far
more than the L2, so every step reads HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl qil|reference]

With N > 1 (launched under torchrun) every rank runs an independent replica on its own GPU
(the path has no cross-GPU exchange); the reported value is the sum over ranks divided by the
slowest rank's time.  ``--impl reference`` times the CPU oracle on a bounded sample instead.
Prints one JSON line on rank 0.
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

METRIC = "W4A16 GEMV GB/s at Llama-2-7B M=1 (packed weights + scales + zeros + activations streamed per second)"
UNIT = "GB/s"
DECODE_PROFILE = os.path.join(ROOT, "profiles", "w4a16_tc_kernel_cfg1_decode.json")
DECODE_KERNEL_SOURCE = os.path.join(ROOT, "paper_2412_01034_b200", "csrc", "w4a16_tc.cu")
WORKLOAD = "configs[1]: Llama-2-7B decoder linears, decode M=1, 32 layers x 7 linears, group 128, 0.1% outliers"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def reduce_max_time_sum_units(ms_local: float, units_local: float, world: int, backend_device):
    """(max over ranks of the time, sum over ranks of the units); identity for one rank."""
    if world == 1:
        return ms_local, units_local
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=backend_device)
    u = torch.tensor([units_local], dtype=torch.float64, device=backend_device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100", "-i", str(index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    @staticmethod
    def _epoch(stamp: str) -> float:
        import datetime
        return datetime.datetime.strptime(stamp, "%Y/%m/%d %H:%M:%S.%f").timestamp()

    def stop(self, t0: float, t1: float):
        """Summary of the samples taken between the host times t0 and t1 (all samples if none fall inside)."""
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for line in out.strip().splitlines():
            f = [p.strip() for p in line.split(",")]
            if len(f) < 8:
                continue
            try:
                rows.append((self._epoch(f[0]), float(f[1]), float(f[2]), float(f[3]),
                             [n for n, v in zip(names, f[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if t0 <= r[0] <= t1]
        use = inside or rows
        if not use:
            return None
        reasons = sorted({n for r in use for n in r[4]})
        return {"sm_mhz": statistics.median(r[1] for r in use), "sm_max_mhz": max(r[2] for r in use),
                "power_w_max": max(r[3] for r in use), "samples": len(use),
                "window": "timed region" if inside else "warm-up and timed region", "reasons": reasons}


def measured_dram_bytes_per_layer():
    """DRAM read + write bytes of the decode kernel per decoder layer, from the tracked summary of its last ncu
    capture; None when the kernel source has changed since that capture (the figure would describe another kernel)."""
    import hashlib
    try:
        prof = json.load(open(DECODE_PROFILE))
        digest = hashlib.sha256(open(DECODE_KERNEL_SOURCE, "rb").read()).hexdigest()
    except (OSError, ValueError):
        return None
    if prof.get("kernel_source_sha256") != digest:
        return None
    return (prof["dram_bytes_read"] + prof["dram_bytes_write"]) / prof["layers_captured"]


def check_against_oracle(model, sampled):
    """After the timed region: the status word of the workspace must be 0 and the sampled output features of the
    sampled linears must match the CPU oracle (quantiser + fp64 linear) within the acceptance rule."""
    import ctypes as C
    import numpy as np
    import torch
    from oracle import c_oracle
    from paper_2412_01034_b200 import workloads as wl
    model.y_dev.zero_()
    model.run()
    torch.cuda.synchronize()
    out = C.c_int(-1)
    rc = model.lib.qil_device_status(C.c_void_p(model.ws.data_ptr()), C.byref(out),
                                     C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc != 0 or out.value != 0:
        raise SystemExit(f"bench: device status word is {out.value} (rc {rc}) after the timed region")
    worst = 0.0
    for i in sampled:
        rows, w_rows = model.kept[i]
        q = c_oracle.quantize_rtn_w4_asym(w_rows, wl.GROUP_SIZE)
        y_ref = c_oracle.linear_w4a16(model.input_bits(i), *q, wl.GROUP_SIZE)
        y = model.output(i).to(torch.float32).cpu().numpy().astype(np.float64)[:, rows]
        # (the maximum over the sampled features lower-bounds the row maximum: the check is the stricter one)
        rel = float((np.abs(y - y_ref) / np.abs(y_ref).max(axis=1, keepdims=True)).max())
        worst = max(worst, rel)
        if not np.all(np.isfinite(y)) or rel > 1e-2:
            raise SystemExit(f"bench: linear {i} differs from the oracle (row-relative error {rel:.3e})")
    return worst


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            pass
    return local_rank


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample(budget_s: float, max_layers: int):
    """Times the plain-C oracle's dequantise-then-matmul (fp64) on whole decoder layers of the same
    workload until about ``budget_s`` seconds of CPU work are done.  Returns (GB/s, cores, description)."""
    from oracle import c_oracle
    from paper_2412_01034_b200 import workloads as wl
    specs = wl.llama_linear_ids()
    done_bytes, spent, layers = 0, 0.0, 0
    per_layer = len(wl.LLAMA2_7B_LAYER)
    while layers < max_layers and spent < budget_s:
        for (_, _, N, K, tw, tx) in specs[layers * per_layer:(layers + 1) * per_layer]:
            w = wl.llama_weight(1, tw, N, K)
            codes, s, z = c_oracle.quantize_rtn_w4_asym(w, wl.GROUP_SIZE)   # setup, not timed
            x = wl.normal_activations_bf16(1, tx, 1, K)
            t0 = time.perf_counter()
            c_oracle.linear_w4a16(x, codes, s, z, wl.GROUP_SIZE)
            spent += time.perf_counter() - t0
            done_bytes += N * K // 2 + 4 * N * (K // wl.GROUP_SIZE) + 2 * K + 2 * N
        layers += 1
    return done_bytes / spent / 1e9, c_oracle.num_threads(), f"{layers} of 32 decoder layers ({layers * per_layer} linears), M=1, fp64 C/OpenMP oracle"


def run_reference(args):
    rank, _, _ = dist_env()
    if rank != 0:
        return
    from oracle import c_oracle
    from paper_2412_01034_b200 import workloads as wl
    specs = wl.llama_linear_ids()[:1]   # one linear per step, so that a long --steps run stays bounded
    prepared = []
    for (_, _, N, K, tw, tx) in specs:
        w = wl.llama_weight(1, tw, N, K)
        prepared.append((wl.normal_activations_bf16(1, tx, 1, K), *c_oracle.quantize_rtn_w4_asym(w, wl.GROUP_SIZE)))
    nbytes = sum(N * K // 2 + 4 * N * (K // wl.GROUP_SIZE) + 2 * K + 2 * N for (_, _, N, K, _, _) in specs)

    def step():
        for (x, codes, s, z) in prepared:
            c_oracle.linear_w4a16(x, codes, s, z, wl.GROUP_SIZE)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    ms = (time.perf_counter() - t0) * 1e3 / args.steps
    value = nbytes / (ms * 1e-3) / 1e9
    sample = "layer 0 q projection (4096 x 4096, 16.8 M weights) per step, M=1, fp64 C/OpenMP oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": c_oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
def run_qil(args):
    import torch
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2412_01034_b200 import api, llama_decode

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, sample = oracle_sample(args.cpu_budget_s, 32)
        cpu_baseline = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}

    layout = {"stream128": api.LAYOUT_STREAM128, "tile16": api.LAYOUT_TILE16,
              "canonical": api.LAYOUT_CANONICAL}[args.layout]
    persistent = args.layout == "stream128"
    import numpy as np
    per_layer = 7
    sampled = sorted({0, (args.layers // 2) * per_layer + 4, (args.layers - 1) * per_layer + 6})   # a q, a gate, a down
    rng = np.random.default_rng(5)
    keep = {}
    from paper_2412_01034_b200 import workloads as wl
    for i in sampled:
        keep[i] = np.sort(rng.choice(wl.llama_linear_ids()[i][2], 64, replace=False))
    model = llama_decode.QuantisedLinears(cfg=1, M=1, n_layers=args.layers, layout=layout, deps=args.deps,
                                          device=f"cuda:{local_rank}", keep_host_rows=keep)
    stream = torch.cuda.Stream(device=dev)
    bytes_per_step = model.algorithmic_bytes()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn(stream)                      # eager once (also sets kernel attributes outside capture)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                fn(stream)
        return g

    def timed(graph, steps, warmup, sampler_index=None):
        with torch.cuda.stream(stream):
            sampler = ClockSampler(sampler_index) if sampler_index is not None else None
            for _ in range(warmup):
                graph.replay()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.time()
            e0.record(stream)
            for _ in range(steps):
                graph.replay()
            e1.record(stream)
            barrier()
            t1 = time.time()
            clocks = sampler.stop(t0, t1) if sampler else None
        return e0.elapsed_time(e1) / steps, clocks

    g_dev = capture(lambda s: model.run(s))
    g_e2e = capture(lambda s: model.run_host(s))

    ms, clocks = timed(g_dev, args.steps, args.warmup, physical_gpu_index(local_rank) if rank == 0 else None)
    ms_e2e, _ = timed(g_e2e, args.steps, args.warmup)

    parity_worst = check_against_oracle(model, sampled)

    ms_all, units_all = reduce_max_time_sum_units(ms, bytes_per_step, world, dev)
    ms_e2e_all, _ = reduce_max_time_sum_units(ms_e2e, bytes_per_step, world, dev)
    value = units_all / (ms_all * 1e-3) / 1e9
    value_e2e = units_all / (ms_e2e_all * 1e-3) / 1e9

    n_linears, x_elems, y_elems = model.count, model.x_elems, model.y_elems
    secondary = None
    ordered = None
    if rank == 0 and world == 1 and not args.no_secondary and persistent and args.deps == "none":
        # the same list with the linears ordered as a decoder layer orders them (each wait is a grid-wide hand-over)
        model.set_deps("layer")
        g_ord = capture(lambda s: model.run(s))
        ms_ord, _ = timed(g_ord, min(args.steps, 200), min(args.warmup, 20))
        ordered = {"dependencies": "layer", "ms_per_step": ms_ord, "GB/s": bytes_per_step / (ms_ord * 1e-3) / 1e9,
                   "waiting_linears_per_step": sum(1 for i in range(n_linears) if model.descs[i].flags)}
        ordered["parity_worst_row_relative_error"] = check_against_oracle(model, sampled)
        model.set_deps("none")
        del g_ord
    if rank == 0 and world == 1 and not args.no_secondary:
        del g_dev, g_e2e, model
        torch.cuda.empty_cache()
        secondary = secondary_measurements(dev)
        if ordered is not None:
            secondary["w4a16_decode_in_decoder_layer_order"] = ordered

    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except (OSError, ValueError):
            pass
        peak = float(peaks.get("hbm_gbs", 6650.0))
        peak_kind = "measured copy bandwidth (MEASURED_PEAKS.json)" if "hbm_gbs" in peaks else "fallback 6650 GB/s"
        launches_per_step = 1 if persistent else n_linears
        kernel = "w4a16_tc_kernel<1>" if persistent else "w4a16_skinny_kernel<1>"
        per_launch_bytes = bytes_per_step / launches_per_step
        per_launch_ms = ms / launches_per_step          # average over the timed region, launch gaps included
        achieved = per_launch_bytes / (per_launch_ms * 1e-3) / 1e9
        # dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of this kernel on 2 layers (14 independent
        # linears, larger than L2): 110.16 MB per layer, scaled by the layers of a launch (traffic grows in proportion)
        per_layer_traffic = measured_dram_bytes_per_layer() if (persistent and args.deps == "none") else None
        traffic = per_layer_traffic * args.layers if per_layer_traffic else None
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_all, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 activations x int4 weights, fp32 accumulate", "data": "synthetic",
            "config": {"workload": WORKLOAD, "layers": args.layers, "linears_per_step": n_linears,
                       "layout": args.layout, "dependencies": args.deps,
                       "bytes_per_step": bytes_per_step, "l2": "inputs larger than L2 (3.44 GB of weights per step)",
                       "parallelism": f"replicas x{world}", "launch": ("CUDA graph of one persistent kernel over the whole list" if persistent
                                  else "CUDA graph of one kernel per linear")},
            "clocks": clocks,
            "e2e": {"value": value_e2e, "unit": UNIT, "ms_per_step": ms_e2e_all,
                    "h2d_bytes_per_step": 2 * x_elems, "d2h_bytes_per_step": 2 * y_elems},
            "gpu_launches": launches_per_step * args.steps,
            "parity_checked": True,
            "parity": {"status_word": 0, "linears": sampled, "features_per_linear": 64,
                       "worst_row_relative_error": parity_worst, "bound": 1e-2},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_kind": peak_kind, "kernel": kernel,
                         "bytes_per_launch": per_launch_bytes, "us_per_launch": per_launch_ms * 1e3,
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "cpu_baseline": cpu_baseline,
            "secondary": secondary,
        }
        print(json.dumps(out))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def secondary_measurements(dev):
    """Short timings of the other rows of the path on the same GPU (each a few milliseconds): the W4A4 integer
    GEMM on the four im2col conv shapes (GEMM alone and with the per-token activation quantiser), the 16-bit
    reference GEMV the 4-bit decode is compared with, and one decoder layer at prefill length 280."""
    import numpy as np
    import torch
    from paper_2412_01034_b200 import api, workloads as wl
    out = {}

    def time_us(fn, reps):
        """Device time per call: `reps` calls captured in a CUDA graph (these kernels are shorter than a launch
        from Python), the graph replayed three times and timed with events on its stream."""
        st = torch.cuda.Stream(device=dev)
        with torch.cuda.stream(st):
            for _ in range(3):
                fn()
            st.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                for _ in range(reps):
                    fn()
            graph.replay()
            st.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(3):
                graph.replay()
            e1.record(st)
            st.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (3 * reps)

    g = torch.Generator(device=dev)
    g.manual_seed(4)

    def time_event_us(fn):
        """One launch timed with events on the current stream (for launches of tens of microseconds or more)."""
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3

    # roofs measured by the library's own probes: a read-only pass over 2 GiB (a GEMV reads, it does not copy) and
    # tcgen05.mma over operands resident in shared memory
    buf = torch.empty(1 << 29, dtype=torch.int32, device=dev)
    sink = torch.zeros(1, dtype=torch.int32, device=dev)
    t_read = min(time_event_us(lambda: api.probe_hbm_read(buf, sink)) for _ in range(3))
    del buf
    pstat = torch.zeros(4, dtype=torch.int32, device=dev)
    probes = {"hbm_read_GB/s": (1 << 31) / t_read / 1e3}
    for kind, key in (("i8", "mma_i8_TOPS"), ("bf16", "mma_bf16_TFLOP/s")):
        ops = api.probe_mma(kind, 2000, 8, status=pstat)
        t = min(time_event_us(lambda: api.probe_mma(kind, 2000, 8, status=pstat)) for _ in range(3))
        probes[key] = ops / t / 1e6
    probes["status"] = int(pstat[0].item())
    probes["note"] = "burst figures: each probe launch lasts well under a millisecond"
    out["probes"] = probes
    i8_roof = probes["mma_i8_TOPS"]

    conv, conv8 = [], []
    l2_bytes = 126 * 1024 * 1024
    for stage in range(4):
        M, K, N = wl.conv_gemm_shape(stage)
        x = torch.relu(torch.randn((M, K), device=dev, generator=g)).to(torch.bfloat16)
        w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_CONV
        qw, sw, _ = api.quantize_rtn_w4(w, K, symmetric=True)
        pw = api.pack_w4(qw)
        qx, sx = api.quantize_act_a4(x)
        ws = api.new_workspace(api.linear_w4a4_workspace_size(M, N, K), dev)
        y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        t_gemm = time_us(lambda: api.linear_w4a4(qx, sx, pw, sw.reshape(-1), out=y, workspace=ws), 50)
        t_both = time_us(lambda: api.linear_w4a4(*api.quantize_act_a4(x), pw, sw.reshape(-1), out=y, workspace=ws), 50)
        # tensor-wise static activation scale (the paper's W4A4 setting, App. A.1.2): quantiser + GEMM
        t_static = time_us(lambda: api.linear_w4a4(*api.quantize_act_a4(x, static_scale=0.5), pw, sw.reshape(-1), out=y, workspace=ws), 50)
        # cold: distinct operand and output copies in rotation, together more than four times the L2
        per_copy = M * K // 2 + N * K // 2 + 2 * M * N + 4 * (M + N)
        copies = min(160, 4 * l2_bytes // per_copy + 1)
        qxs = [qx.clone() for _ in range(copies)]
        pws = [pw.clone() for _ in range(copies)]
        ys = [torch.empty_like(y) for _ in range(copies)]
        st_ = {"i": 0}

        def cold():
            i = st_["i"] % copies
            st_["i"] += 1
            api.linear_w4a4(qxs[i], sx, pws[i], sw.reshape(-1), out=ys[i], workspace=ws)
        t_cold = time_us(cold, copies)
        del qxs, pws, ys
        ops = 2.0 * M * K * N
        conv.append({"M": M, "K": K, "N": N, "gemm_us": t_gemm, "gemm_tops": ops / t_gemm / 1e6,
                     "gemm_cold_us": t_cold, "gemm_cold_tops": ops / t_cold / 1e6,
                     "quantise_plus_gemm_us": t_both, "static_scale_quantise_plus_gemm_us": t_static,
                     "frac_of_i8_probe": ops / t_gemm / 1e6 / i8_roof,
                     "l2": "warm: operands resident in L2; cold: %d copies in rotation" % copies})
        # the same shapes with 8-bit operands (Table "CILRS performance", W8A8 row)
        qw8, sw8, _ = api.quantize_rtn_w8(w, K, symmetric=True)
        qx8, sx8 = api.quantize_act_a8(x)
        t8 = time_us(lambda: api.linear_w8a8(qx8, sx8, qw8, sw8.reshape(-1), out=y, workspace=ws), 50)
        t8_both = time_us(lambda: api.linear_w8a8(*api.quantize_act_a8(x), qw8, sw8.reshape(-1), out=y, workspace=ws), 50)
        conv8.append({"M": M, "K": K, "N": N, "gemm_us": t8, "gemm_tops": ops / t8 / 1e6, "quantise_plus_gemm_us": t8_both,
                      "frac_of_i8_probe": ops / t8 / 1e6 / i8_roof})
    # the four GEMMs (independent operands) as one persistent launch
    for bits_, key in ((4, "w4a4_conv_stages_one_launch"), (8, "w8a8_conv_stages_one_launch")):
        ents, ops_all = [], 0.0
        for stage in range(4):
            M, K, N = wl.conv_gemm_shape(stage)
            x = torch.relu(torch.randn((M, K), device=dev, generator=g)).to(torch.bfloat16)
            w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_CONV
            if bits_ == 4:
                qw_, sw_, _ = api.quantize_rtn_w4(w, K, symmetric=True)
                qw_ = api.pack_w4(qw_)
                qx_, sx_ = api.quantize_act_a4(x)
            else:
                qw_, sw_, _ = api.quantize_rtn_w8(w, K, symmetric=True)
                qx_, sx_ = api.quantize_act_a8(x)
            ents.append((qx_, sx_, qw_, sw_.reshape(-1), torch.empty((M, N), dtype=torch.bfloat16, device=dev), None, bits_))
            ops_all += 2.0 * M * K * N
        wsl = api.new_workspace(16, dev)
        t_l = time_us(lambda: api.linear_int_batch(ents, workspace=wsl), 50)
        out[key] = {"us": t_l, "tops": ops_all / t_l / 1e6, "frac_of_i8_probe": ops_all / t_l / 1e6 / i8_roof,
                    "kernel": "igemm_list_kernel", "l2": "warm"}
    # the same four layers read straight from int4 feature maps (no im2col matrix), bf16 output and int4 output
    fm = []
    for stage in range(4):
        Cc, H, W = wl.CONV_STAGES[stage]
        B = wl.CONV_BATCH
        codes = torch.randint(-8, 8, (B * H * W, Cc), device=dev, generator=g, dtype=torch.int32).to(torch.int8)
        qf = api.pack_w4(codes).reshape(B, H, W, Cc // 8)
        w = torch.randn((Cc, 9 * Cc), device=dev, generator=g) * wl.SIGMA_CONV
        qw_, sw_, _ = api.quantize_rtn_w4(w, 9 * Cc, symmetric=True)
        pw_ = api.pack_w4(qw_)
        wsc = api.new_workspace(api.linear_w4a4_workspace_size(B * H * W, Cc, 9 * Cc), dev)
        t_bf = time_us(lambda: api.conv3x3_w4a4(qf, 0.25, pw_, sw_.reshape(-1), workspace=wsc), 50)
        t_q = time_us(lambda: api.conv3x3_w4a4(qf, 0.25, pw_, sw_.reshape(-1), out_scale=0.5, relu=True, workspace=wsc), 50)
        ops = 2.0 * B * H * W * 9 * Cc * Cc
        fm.append({"C": Cc, "H": H, "W": W, "batch": B, "bf16_out_us": t_bf, "int4_out_us": t_q, "tops": ops / t_q / 1e6})
    out["w4a4_conv3x3_from_feature_map"] = fm
    out["w4a4_conv3x3_from_feature_map_tops_total"] = sum(2.0 * f["batch"] * f["H"] * f["W"] * 9 * f["C"] ** 2 for f in fm) / sum(f["int4_out_us"] for f in fm) / 1e6
    out["w4a4_conv_stages"] = conv
    out["w4a4_tops_total"] = sum(2.0 * c["M"] * c["K"] * c["N"] for c in conv) / sum(c["gemm_us"] for c in conv) / 1e6
    out["w4a4_tops_total_cold"] = sum(2.0 * c["M"] * c["K"] * c["N"] for c in conv) / sum(c["gemm_cold_us"] for c in conv) / 1e6
    out["w8a8_conv_stages"] = conv8
    out["w8a8_tops_total"] = sum(2.0 * c["M"] * c["K"] * c["N"] for c in conv8) / sum(c["gemm_us"] for c in conv8) / 1e6

    # the policy MLP of the DM-Control / D4RL experiments (Sec. 5.1: three fully connected layers of 2048 units) as
    # W4A4: per-token activation quantiser + integer GEMM per layer, a latency case
    mlp = []
    wq = []
    for _ in range(3):
        w = torch.randn((2048, 2048), device=dev, generator=g) * wl.SIGMA_CONV
        qw, sw, _ = api.quantize_rtn_w4(w, 2048, symmetric=True)
        wq.append((api.pack_w4(qw), sw.reshape(-1)))
    for Mb in (1, 256):
        xin = torch.randn((Mb, 2048), device=dev, generator=g).to(torch.bfloat16)
        bufs = [torch.empty((Mb, 2048), dtype=torch.bfloat16, device=dev) for _ in range(3)]
        ws = api.new_workspace(api.linear_w4a4_workspace_size(Mb, 2048, 2048), dev)

        def mlp_pass():
            cur = xin
            for (pw_, sw_), yb in zip(wq, bufs):
                api.linear_w4a4(*api.quantize_act_a4(cur), pw_, sw_, out=yb, workspace=ws)
                cur = yb
        t = time_us(mlp_pass, 20)
        mlp.append({"batch": Mb, "us_per_pass": t, "layers": 3, "units": 2048})
    out["w4a4_policy_mlp_3x2048"] = mlp

    # the paper's channel-wise weight setting (App. A.1.2: group_size = K) on one 4096 x 4096 decode linear, cold
    N = K = wl.HIDDEN
    copies = 12
    chan = []
    for _ in range(copies):
        w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_LLM
        codes, s_, z_ = api.quantize_rtn_w4(w, K)
        chan.append(api.pack_stream128_w4(codes, s_, z_, K))
        del w, codes
    xv1 = torch.randn((1, K), device=dev, generator=g).to(torch.bfloat16)
    yv1 = torch.empty((1, N), dtype=torch.bfloat16, device=dev)
    wsc = api.new_workspace(api.linear_w4a16_workspace_size(1, N, K, K), dev)
    stc = {"i": 0}

    def chan_one():
        api.linear_w4a16(xv1, chan[stc["i"] % copies], None, None, N, K, api.LAYOUT_STREAM128, out=yv1, workspace=wsc)
        stc["i"] += 1
    t_chan = time_us(chan_one, 4 * copies)
    out["w4a16_channelwise_4096x4096_m1"] = {"us": t_chan, "GB/s": (N * K / 2 + 4 * N + 2 * K + 2 * N) / t_chan / 1e3,
                                             "l2": f"cold: {copies} weight copies in rotation", "note": "single call: includes the start-up of one launch"}
    del chan

    # INT8 weight-only decode (Table "OpenVLA performance", INT8 row): 8 decoder layers of the Llama-2-7B list
    # (1.6 GB of codes, larger than L2) in one launch of the 8-bit streaming kernel
    from paper_2412_01034_b200 import llama_decode
    m8 = llama_decode.QuantisedLinears(cfg=1, M=1, n_layers=8, deps="none", device=str(dev), bits=8)
    st8 = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(st8):
        for _ in range(3):
            m8.run(st8)
        st8.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st8)
        for _ in range(20):
            m8.run(st8)
        e1.record(st8)
        st8.synchronize()
    t8l = e0.elapsed_time(e1) / 20
    w8 = {"layers": 8, "ms_per_pass": t8l, "GB/s": m8.algorithmic_bytes() / (t8l * 1e-3) / 1e9,
          "bytes_per_pass": m8.algorithmic_bytes(), "kernel": "w8a16_stream_kernel<1> (dp4a)"}
    m8.set_deps("layer")
    with torch.cuda.stream(st8):
        m8.run(st8)
        st8.synchronize()
        e0.record(st8)
        for _ in range(20):
            m8.run(st8)
        e1.record(st8)
        st8.synchronize()
    w8["decoder_layer_order_GB/s"] = m8.algorithmic_bytes() / (e0.elapsed_time(e1) / 20 * 1e-3) / 1e9
    out["w8a16_decode_list"] = w8
    del m8

    # 16-bit reference GEMV, cold: rotate over copies larger than L2
    N = K = wl.HIDDEN
    copies = 12
    wd = [torch.randn((N, K), device=dev, generator=g).to(torch.bfloat16) for _ in range(copies)]
    xv = torch.randn((1, K), device=dev, generator=g).to(torch.bfloat16)
    yv = torch.empty((N,), dtype=torch.bfloat16, device=dev)
    state = {"i": 0}

    def ref():
        api.ref_gemv_bf16(xv, wd[state["i"] % copies], out=yv)
        state["i"] += 1
    t_ref = time_us(ref, 48)
    out["ref_gemv_bf16_4096x4096"] = {"us": t_ref, "GB/s": (2.0 * N * K + 2 * K + 2 * N) / t_ref / 1e3,
                                      "l2": f"cold: {copies} weight copies in rotation"}
    del wd

    # prefill: one decoder layer (7 linears) at M = 280
    Mp = wl.PREFILL_M
    xs = {K: torch.randn((Mp, K), device=dev, generator=g).to(torch.bfloat16) for K in (wl.HIDDEN, wl.FFN)}
    lin = []
    for (_, N, K) in wl.LLAMA2_7B_LAYER:
        w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_LLM
        codes, s, z = api.quantize_rtn_w4(w, wl.GROUP_SIZE)
        lin.append((N, K, api.pack_w4(codes), s, z, torch.empty((Mp, N), dtype=torch.bfloat16, device=dev),
                    api.new_workspace(api.linear_w4a16_workspace_size(Mp, N, K, wl.GROUP_SIZE), dev)))
        del w, codes

    def layer():
        for (N, K, pk, s, z, yo, ws) in lin:
            api.linear_w4a16(xs[K], pk, s, z, N, wl.GROUP_SIZE, api.LAYOUT_CANONICAL, out=yo, workspace=ws)
    t_layer = time_us(layer, 10)
    del lin

    # the same layer with q, k, v and gate, up stored as one linear each (4 launches instead of 7)
    linf = []
    for (_, N, K) in wl.LLAMA2_7B_LAYER_FUSED:
        w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_LLM
        codes, s, z = api.quantize_rtn_w4(w, wl.GROUP_SIZE)
        linf.append((N, K, api.pack_w4(codes), s, z, torch.empty((Mp, N), dtype=torch.bfloat16, device=dev),
                     api.new_workspace(api.linear_w4a16_workspace_size(Mp, N, K, wl.GROUP_SIZE), dev)))
        del w, codes

    def layer_fused():
        for (N, K, pk, s, z, yo, ws) in linf:
            api.linear_w4a16(xs[K], pk, s, z, N, wl.GROUP_SIZE, api.LAYOUT_CANONICAL, out=yo, workspace=ws)
    t_layer_fused = time_us(layer_fused, 10)
    # the gate_up linear alone, plain and with silu(gate) * up in its epilogue (the same rows read as interleaved pairs)
    (Ng, Kg, pkg, sg, zg, yg, wsg) = linf[2]
    ysw = torch.empty((Mp, Ng // 2), dtype=torch.bfloat16, device=dev)
    wsw = api.new_workspace(api.linear_w4a16_swiglu_workspace_size(Mp, Ng, Kg, wl.GROUP_SIZE), dev)
    t_gate_up = time_us(lambda: api.linear_w4a16(xs[Kg], pkg, sg, zg, Ng, wl.GROUP_SIZE, api.LAYOUT_CANONICAL, out=yg, workspace=wsg), 10)
    t_gate_up_sw = time_us(lambda: api.linear_w4a16_swiglu(xs[Kg], pkg, sg, zg, Ng, wl.GROUP_SIZE, out=ysw, workspace=wsw), 10)
    del linf, xs, ysw, wsw

    # configs[3]: M sweep on the two FFN shapes, cold (6 weight copies in rotation = 144 MB of packed weights,
    # larger than L2).  M <= 4 runs the tcgen05 decode kernel (STREAM128 units), M <= 8 the mma.sync skinny kernel
    # (TILE16), larger M the tcgen05 prefill kernel (canonical layout).
    sweep = []
    copies = 6
    for (N, K) in ((wl.FFN, wl.HIDDEN), (wl.HIDDEN, wl.FFN)):
        packs = {"stream128": [], "tile16": [], "canonical": []}
        sz = []
        for _ in range(copies):
            w = torch.randn((N, K), device=dev, generator=g) * wl.SIGMA_LLM
            codes, s_, z_ = api.quantize_rtn_w4(w, wl.GROUP_SIZE)
            packs["stream128"].append(api.pack_stream128_w4(codes, s_, z_, wl.GROUP_SIZE))
            packs["tile16"].append(api.pack_w4(codes, api.LAYOUT_TILE16))
            packs["canonical"].append(api.pack_w4(codes, api.LAYOUT_CANONICAL))
            sz.append((s_, z_))
            del w, codes
        lay = {"stream128": api.LAYOUT_STREAM128, "tile16": api.LAYOUT_TILE16, "canonical": api.LAYOUT_CANONICAL}
        for Ms in (1, 2, 4, 8, 16, 32, 64, 128, 280):
            xm = torch.randn((Ms, K), device=dev, generator=g).to(torch.bfloat16)
            ym = torch.empty((Ms, N), dtype=torch.bfloat16, device=dev)
            ws = api.new_workspace(api.linear_w4a16_workspace_size(Ms, N, K, wl.GROUP_SIZE), dev)
            for name in (("stream128", "tile16") if Ms <= 4 else ("tile16",) if Ms <= 8 else ("canonical",)):
                st_ = {"i": 0}

                def one():
                    i = st_["i"] % copies
                    st_["i"] += 1
                    if name == "stream128":
                        api.linear_w4a16(xm, packs[name][i], None, None, N, wl.GROUP_SIZE, lay[name], out=ym, workspace=ws)
                    else:
                        api.linear_w4a16(xm, packs[name][i], sz[i][0], sz[i][1], N, wl.GROUP_SIZE, lay[name], out=ym, workspace=ws)
                t = time_us(one, 4 * copies)
                by = N * K * 0.53125 + 2.0 * Ms * K + 2.0 * Ms * N
                sweep.append({"N": N, "K": K, "M": Ms, "layout": name, "us": t, "GB/s": by / t / 1e3,
                              "TFLOP/s": 2.0 * Ms * N * K / t / 1e6})
        del packs, sz
    out["w4a16_m_sweep"] = sweep
    flops = sum(2.0 * Mp * N * K for (_, N, K) in wl.LLAMA2_7B_LAYER)
    out["w4a16_prefill_m280_layer"] = {"us": t_layer, "TFLOP/s": flops / t_layer / 1e6, "kernel": "w4a16_prefill_kernel (tcgen05 kind::f16)"}
    # the unmerged rank-32 adapter beside a 4096 x 4096 linear, at decode and at prefill length
    lora = {}
    for Ml in (1, Mp):
        xl = torch.randn((Ml, wl.HIDDEN), device=dev, generator=g).to(torch.bfloat16)
        al = (torch.randn((32, wl.HIDDEN), device=dev, generator=g) * 0.02).to(torch.bfloat16)
        bl = (torch.randn((wl.HIDDEN, 32), device=dev, generator=g) * 0.02).to(torch.bfloat16)
        yl = torch.zeros((Ml, wl.HIDDEN), dtype=torch.bfloat16, device=dev)
        wsl = api.new_workspace(api.lora_side_workspace_size(Ml), dev)
        lora[f"m{Ml}_us"] = time_us(lambda: api.lora_side_add(xl, al, bl, yl, 1.0, workspace=wsl), 20)
    out["lora_side_rank32_4096x4096"] = lora
    out["w4a16_prefill_m280_gate_up_22016x4096"] = {"plain_us": t_gate_up, "swiglu_epilogue_us": t_gate_up_sw,
                                                    "TFLOP/s": 2.0 * Mp * 2 * wl.FFN * wl.HIDDEN / t_gate_up_sw / 1e6}
    out["w4a16_prefill_m280_layer_fused_qkv_gate_up"] = {"us": t_layer_fused, "TFLOP/s": flops / t_layer_fused / 1e6,
                                                         "linears": [n for (n, _, _) in wl.LLAMA2_7B_LAYER_FUSED]}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1050)
    ap.add_argument("--warmup", type=int, default=70)
    ap.add_argument("--impl", default="qil", choices=["qil", "reference"])
    ap.add_argument("--layers", type=int, default=32, help="decoder layers (32 = the stated workload)")
    ap.add_argument("--layout", default="stream128", choices=["stream128", "tile16", "canonical"])
    ap.add_argument("--deps", default="none", choices=["layer", "all", "none"],
                    help="which linears wait for all earlier ones (none = independent GEMVs, the metric; layer = the "
                         "order a decoder layer imposes, also timed as a secondary measurement)")
    ap.add_argument("--cpu-budget-s", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the short W4A4 / reference / prefill timings")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_qil(args)


if __name__ == "__main__":
    main()
