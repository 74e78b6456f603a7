#!/usr/bin/env python
"""Benchmark of the DiRotQ W4A4 linear layer on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference]

One "step" is one pass of the whole hot path (rotate + split + quantize, W4A4 group GEMM,
rank-r branch, epilogue) over the four FLUX.1-dev-shaped linears at M = 4608 tokens
(3072->9216, 3072->3072, 3072->12288, 12288->3072; r = 32, group 64).  The metric is effective
TOPS, sum(2*M*N*K) / time.  Inputs are seeded and synthetic (see paper_2605_16732_b200/synth.py).

With N > 1 (torchrun) every rank runs the same step on its own M tokens (token rows are
independent: no collective on the data path) and the value is the aggregate over ranks.

``--impl reference`` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

FLUX_SHAPES = [("qkv", 3072, 9216), ("out", 3072, 3072), ("mlp_up", 3072, 12288), ("mlp_down", 12288, 3072)]
M_TOKENS = 4608
RANK, GROUP = 32, 64
WORKLOAD = "flux1dev_linears_M4608_r32_g64"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                          "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        # median over the samples taken under load (upper half by clock x power is a poor proxy; use power)
        order = np.argsort(power)
        load = [sm[i] for i in order[len(order) // 2:]]
        return {"sm_mhz": float(np.median(load)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": float(max(power))}


def _shape_ops(M):
    return sum(2.0 * M * N * K for _, K, N in FLUX_SHAPES)


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (bounded sample)


def oracle_sample_run(steps: int, rows: int = 32, cols: int = 128, seed: int = 0, fmt: str = "int4"):
    """Times the oracle's online steps on `rows` tokens x `cols` output columns of every linear."""
    from oracle import dirotq_oracle as orc
    from paper_2605_16732_b200 import synth

    layers = []
    for name, K, N in FLUX_SHAPES:
        spec = synth.LayerSpec(K=K, N=N, r=RANK, G=GROUP, model=synth.FLUX, seed=seed)
        g = np.random.Generator(np.random.Philox(key=[K, N]))
        # the oracle's run time does not depend on the rotation's values: a seeded Householder
        # reflection (dense, exactly orthogonal) stands in for the PCA rotation, whose
        # eigendecomposition takes minutes on a CPU at K = 12288
        v = g.standard_normal(K)
        v /= np.linalg.norm(v)
        Q = np.eye(K) - 2.0 * np.outer(v, v)
        W = (0.02 * g.standard_normal((K, cols))).astype(np.float32)
        x = synth.make_tokens(spec, rows, batch_seed=5)
        if fmt == "w4a8":
            lo = orc.prepare_layer_w4a8(W, Q, RANK)
        elif fmt == "nvfp4":
            lo = orc.nvfp4_prepare_layer(W, Q, RANK)
            lo["ex"] = orc.nvfp4_global_exponent(float(np.abs(orc.rotate(x, lo["Qb"])[:, RANK:]).max()))
        elif fmt == "int4_ph":
            lo = orc.prepare_layer_ph(W, np.ascontiguousarray(Q[:, :RANK]), GROUP)
        elif fmt == "nvfp4_ph":
            lo = orc.nvfp4_prepare_layer_ph(W, np.ascontiguousarray(Q[:, :RANK]))
            lo["ex"] = orc.nvfp4_global_exponent(float(np.abs(orc.nvfp4_residual(x, lo)[1]).max()))
        else:
            lo = orc.prepare_layer(W, Q, RANK, GROUP)
        layers.append((lo, x, K, cols))
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        for lo, x, K, n in layers:
            if fmt == "nvfp4":
                orc.nvfp4_linear_deployed(x, lo, lo["ex"], bias=None, want_t=False)
            elif fmt == "int4_asym":
                orc.linear_deployed_asym(x, lo, bias=None, want_t=False)
            elif fmt == "w4a8":
                orc.linear_deployed_w4a8(x, lo, bias=None, want_t=False)
            elif fmt == "int4_ph":
                orc.linear_deployed_ph(x, lo, bias=None, want_t=False)
            elif fmt == "nvfp4_ph":
                orc.nvfp4_linear_deployed_ph(x, lo, lo["ex"], bias=None, want_t=False)
            else:
                orc.linear_deployed(x, lo, bias=None, want_t=False)
        times.append(time.perf_counter() - t0)
    ops = sum(2.0 * rows * n * K for _, _, K, n in layers)
    t = float(np.mean(times))
    return {"value": ops / t / 1e12, "unit": "TOPS", "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{rows} token rows x {cols} output columns of each of the 4 linears, online steps only "
                      f"(rotation, quantize, {'block-scaled products' if fmt in ('nvfp4', 'nvfp4_ph') else 'int GEMM'}, combine); Householder rotation",
            "seconds_per_step": t}


def oracle_config1_full():
    """The oracle on the whole PixArt attention-projection layer (M = 256, K = N = 1152, r = 32, groups of 64, PCA rotation of a
    seeded calibration batch): nothing sampled, nothing extrapolated.  Online steps only, best of two runs."""
    from oracle import dirotq_oracle as orc
    from paper_2605_16732_b200 import synth

    spec = synth.LayerSpec(K=1152, N=1152, r=RANK, G=GROUP, model=synth.PIXART, seed=2)
    inp = synth.make_layer_inputs(spec, 256)
    lo = orc.prepare_layer(inp["W"], inp["Q"], RANK, GROUP)
    best = None
    for _ in range(2):
        t0 = time.perf_counter()
        orc.linear_deployed(inp["x"], lo, bias=inp["bias"], want_t=False)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return {"workload": "pixart_attention_projection_M256_K1152_N1152_r32_g64", "seconds": best,
            "value": 2.0 * 256 * 1152 * 1152 / best / 1e12, "unit": "TOPS", "cores": orc.num_threads()}


def _suffix(fmt):
    return {"nvfp4": "_nvfp4", "int4_asym": "_asym", "w4a8": "_w4a8", "int4_ph": "_projection_form",
            "nvfp4_ph": "_projection_form_nvfp4"}.get(fmt, "")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps = max(1, args.steps)
    # the sample shrinks with the number of steps so that the whole run stays within a few minutes of CPU time
    rows, cols = (128, 512) if steps <= 5 else (64, 256) if steps <= 30 else (32, 128)
    for _ in range(min(args.warmup, 1)):
        oracle_sample_run(1, rows=rows, cols=cols, fmt=args.fmt)
    res = oracle_sample_run(steps, rows=rows, cols=cols, fmt=args.fmt)
    line = {
        "impl": "reference", "metric": "dirotq_w4a4_linear_effective_tops", "value": res["value"], "unit": "TOPS",
        "n_gpus": args.gpus, "steps": steps, "warmup": args.warmup, "ms_per_step": res["seconds_per_step"] * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64 (oracle; nvfp4 codes)" if args.fmt in ("nvfp4", "nvfp4_ph") else "f64 + int32 (oracle; int4 codes)",
        "data": "synthetic", "config": {"workload": WORKLOAD + _suffix(args.fmt),
                                        "format": args.fmt,
                                        "sample": res["sample"]},
        "cpu_baseline": {k: res[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": res["value"], "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# CUDA arm


def run_ours(args):
    import torch
    from paper_2605_16732_b200 import binding as dq
    from paper_2605_16732_b200 import synth
    from paper_2605_16732_b200.shard import aggregate_throughput, max_over_ranks

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)

    M = M_TOKENS
    peaks = _peaks()

    def bf(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)

    layers = []
    for name, K, N in FLUX_SHAPES:
        spec = synth.LayerSpec(K=K, N=N, r=RANK, G=GROUP, model=synth.FLUX, seed=100)
        Q = torch.from_numpy(synth.make_rotation(spec, device=str(dev))).to(dev)
        W, bias = synth.make_weights(spec)
        x_bits = synth.make_tokens(spec, M, batch_seed=1000 + rank)
        x = bf(x_bits)
        if args.fmt == "nvfp4":
            # the activations' power-of-two scale is a calibration constant: taken here from this batch's first
            # 1024 tokens, rotated by the library itself (a throw-away layer with exponent 0)
            probe = dq.dirotq_prepare_layer_nvfp4(torch.from_numpy(W).to(dev), Q, RANK, 0, bias=bf(bias))
            xrot = torch.empty((1024, K), dtype=torch.float32, device=dev)
            dq.dirotq_rotate_quantize(x[:1024], probe, dq.alloc_workspace(probe, 1024), xrot)
            ex = dq.dirotq_act_scale_log2_from_rotated(xrot, RANK)
            probe.close()
            del xrot
            layer = dq.dirotq_prepare_layer_nvfp4(torch.from_numpy(W).to(dev), Q, RANK, ex, bias=bf(bias))
        elif args.fmt == "w4a8":
            layer = dq.dirotq_prepare_layer_w4a8(torch.from_numpy(W).to(dev), Q, RANK, bias=bf(bias))
        elif args.fmt == "int4_asym":
            layer = dq.dirotq_prepare_layer_asym(torch.from_numpy(W).to(dev), Q, RANK, GROUP, bias=bf(bias))
        elif args.fmt == "int4_ph":
            layer = dq.dirotq_prepare_layer_ph(torch.from_numpy(W).to(dev), Q[:, :RANK].contiguous(), GROUP, bias=bf(bias))
        elif args.fmt == "nvfp4_ph":
            Uh = Q[:, :RANK].contiguous()
            layer = dq.dirotq_prepare_layer_nvfp4_ph(torch.from_numpy(W).to(dev), Uh, dq.dirotq_act_scale_log2_ph(x[:1024].contiguous(), Uh), bias=bf(bias))
        else:
            layer = dq.dirotq_prepare_layer(torch.from_numpy(W).to(dev), Q, RANK, GROUP, bias=bf(bias))
        del Q
        y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        ws = dq.alloc_workspace(layer, M)
        layers.append({"name": name, "K": K, "N": N, "layer": layer, "x": x, "y": y, "ws": ws, "x_bits": x_bits})
    torch.cuda.synchronize()

    def step():
        for L in layers:
            dq.dirotq_linear(L["x"], L["layer"], L["y"], L["ws"])

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0 and not args.lite:
        sampler.start()
        time.sleep(1.0)
    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    # ---- headline: K steps, device-timed
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    barrier()
    ms_total = max_over_ranks(e0.elapsed_time(e1), dev)
    ms_step = ms_total / args.steps

    # ---- per-kernel durations over the same steps (events on the launching stream)
    evs = []
    for _ in range(args.steps):
        for L in layers:
            a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record()
            dq.dirotq_rotate_quantize(L["x"], L["layer"], L["ws"])
            b.record()
            dq.dirotq_w4a4_gemm(M, L["layer"], L["ws"], L["y"])
            c.record()
            evs.append((L["name"], a, b, c))
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 and not args.lite else None
    per = {}
    for name, a, b, c in evs:
        d = per.setdefault(name, {"rotate_ms": [], "gemm_ms": []})
        d["rotate_ms"].append(a.elapsed_time(b))
        d["gemm_ms"].append(b.elapsed_time(c))
    for L in layers:
        assert dq.dirotq_workspace_status(L["ws"]) == 0, "a device-side wait timed out"

    # ---- measured tensor-pipe rates of this GPU, in this run, taken AFTER the timed regions so that they do not warm the
    # chip ahead of them (the library's own issue-rate probe on operands resident in
    # shared memory: int8 -> int32, bf16 -> fp32, E4M3 -> fp32), and the library int8 GEMM torch exposes
    peak_probe = None
    if rank == 0 and not args.lite:
        peak_probe = {name: dq.dirotq_mma_rate_probe(kind) for kind, name in ((0, "i8_tops"), (1, "bf16_tflops"), (2, "e4m3_tops"))}
        try:
            a8 = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device=dev)
            for _ in range(3):
                torch._int_mm(a8, a8)
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            for _ in range(10):
                torch._int_mm(a8, a8)
            t1.record()
            torch.cuda.synchronize()
            peak_probe["int8_library_gemm_8192_tops"] = 10 * 2.0 * 8192 ** 3 / (t0.elapsed_time(t1) * 1e-3) / 1e12
            del a8
        except Exception as exc:  # not every build of the library GEMM has an int8 path
            peak_probe["int8_library_gemm_8192_tops"] = None
            peak_probe["int8_library_gemm_note"] = str(exc)[:120]

    # ---- cuBLAS bf16 comparison on the same shapes (context)
    cublas = {}
    for L in ([] if args.lite else layers):
        Wb = torch.randn((L["K"], L["N"]), device=dev, dtype=torch.bfloat16) * 0.02
        for _ in range(3):
            torch.matmul(L["x"], Wb)
        ts = []
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); torch.matmul(L["x"], Wb); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        cublas[L["name"]] = float(np.median(ts))
        del Wb

    # ---- end to end through the host entry point (pinned host buffers, copies inside the timed region)
    host = []
    for L in ([] if args.lite else layers):
        xh = torch.empty((M, L["K"]), dtype=torch.bfloat16).pin_memory()
        xh.copy_(L["x"].cpu())
        yh = torch.empty((M, L["N"]), dtype=torch.bfloat16).pin_memory()
        host.append((xh, yh))
    e2e_steps = max(1, min(args.steps, 5))

    # the four linears of a step are independent here (own inputs, outputs, staging buffers and workspaces): each goes on
    # a stream of its own, so one layer's device-to-host copy overlaps the next one's host-to-device copy and kernels
    lane_streams = [torch.cuda.Stream(device=dev) for _ in layers]

    def e2e_step():
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        for L, (xh, yh), st in zip(layers, host, lane_streams):
            st.wait_event(fork)
            dq.dirotq_linear_host(xh, L["layer"], yh, L["x"], L["y"], L["ws"], stream=st)
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    e2e_ms = float("nan")
    if not args.lite:
        e2e_step()
        barrier()
        e0.record()
        for _ in range(e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps, dev)
    h2d = sum(M * L["K"] * 2 for L in layers)
    d2h = sum(M * L["N"] * 2 for L in layers)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ops_step = _shape_ops(M)
    value = aggregate_throughput(ops_step, ms_step, world) / 1e12

    # ---- roofline of the dominant kernel: the rotation GEMM (bf16 tensor cores)
    rot_ms = {n: float(np.mean(v["rotate_ms"])) for n, v in per.items()}
    gemm_ms = {n: float(np.mean(v["gemm_ms"])) for n, v in per.items()}
    rot_total, gemm_total = sum(rot_ms.values()), sum(gemm_ms.values())
    ph = args.fmt in ("int4_ph", "nvfp4_ph")
    # kernels per layer: first kernel + second kernel; W4A8 quantizes in a pass of its own; the projection form's first
    # stage is two passes, plus the kernel that adds up the split reduction when there are few row tiles per SM
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    launches_per_layer = 3 if args.fmt == "w4a8" else (3 + (1 if sm_count // -(-M // 128) > 1 else 0)) if ph else 2
    # projection form: two skinny GEMMs on a 64-wide padded rank instead of the K x K rotation; all K columns are 4-bit
    rot_flops = {n: (4.0 * M * K * 64 if ph else 2.0 * M * K * K) for n, K, _ in FLUX_SHAPES}
    gemm_ops = {n: 2.0 * M * (K if ph else K - RANK) * N for n, K, N in FLUX_SHAPES}
    nv = args.fmt in ("nvfp4", "nvfp4_ph")
    # The measured bf16 figure that applies: the burst one for a timed region of well under a second (clocks at their
    # maximum), the sustained one for a long run under the power cap.
    region_s = ms_total * 1e-3
    regime = "burst" if region_s < 1.5 else "sustained"
    bf16_peak = peaks["bf16_burst"] if regime == "burst" else peaks["bf16_sustained"]
    # nominal ratios of the part: 8-bit (int8 / fp8) 2x and fp4 4x the dense bf16 rate (4.5 and 9 : 2.25 PFLOP/s)
    int8_nominal_ratio_peak = (4.0 if nv else 2.0) * bf16_peak
    # the low-precision peak the fractions below are quoted against: this run's probe of the kernel's own instruction
    # kind where there is one (E4M3 for the exact-integer W4A4 path, int8 for W4A8), else the nominal ratio
    probe_key = None if nv else ("i8_tops" if args.fmt == "w4a8" else "e4m3_tops")
    if peak_probe and probe_key:
        int8_peak, int8_peak_source = peak_probe[probe_key], f"this run's tcgen05 issue-rate probe ({probe_key})"
    else:
        int8_peak = int8_nominal_ratio_peak
        int8_peak_source = f"{'4' if nv else '2'} x {peaks['source']} bf16 {regime} (nominal ratio)"
    # DRAM bytes of one launch of the dominant kernel, from the ncu capture summarised under profiles/
    # (qkv shape; read + write).  Static: a profiler is never run inside the benchmark.
    # one launch each, on the qkv shape (3072 -> 9216, M = 4608); other shapes' launches were not captured
    NCU_TRAFFIC_QKV = {"w4a4_gemm_kernel": 72.8e6, "rotate_quant_kernel": 48.5e6, "nvfp4_gemm_kernel": 57.0e6}
    sm_hz = (clocks or {}).get("sm_mhz") or 1850.0
    elem_steps = sum(M * N * (-(-(K - RANK) // GROUP)) for _, K, N in FLUX_SHAPES)
    alu_peak = 148 * (128.0 / 2.0) * sm_hz * 1e6  # element-steps/s: 2 fused multiply-adds each, 128 fp32 lanes per SM
    if rot_total >= gemm_total:
        ach = sum(rot_flops.values()) / (rot_total * 1e-3) / 1e12
        roofline = {"kernel": "rotate_quant_kernel", "bound": "tensor", "achieved": ach, "peak": bf16_peak,
                    "unit": "TFLOP/s", "frac": ach / bf16_peak, "traffic": NCU_TRAFFIC_QKV["rotate_quant_kernel"],
                    "traffic_note": "ncu dram read+write of one qkv-shaped launch",
                    "peak_source": f"{peaks['source']} bf16 {regime} (timed region {region_s:.2f} s)"}
    else:
        ach = sum(gemm_ops.values()) / (gemm_total * 1e-3) / 1e12
        ach_alu = elem_steps / (gemm_total * 1e-3)
        gname = "nvfp4_gemm_kernel" if nv else "w4a8_gemm_kernel" if args.fmt == "w4a8" else "w4a4_gemm_kernel"
        roofline = {"kernel": gname, "bound": "tensor", "achieved": ach, "peak": int8_peak, "unit": "TOP/s",
                    "frac": ach / int8_peak, "traffic": NCU_TRAFFIC_QKV.get(gname),
                    "traffic_note": "ncu dram read+write of ONE launch on the qkv shape (algorithmic bytes of that launch: 117.5e6); "
                                    "`achieved` is over all four shapes' launches",
                    "peak_source": int8_peak_source,
                    "achieved_qkv_launch": gemm_ops["qkv"] / (gemm_ms["qkv"] * 1e-3) / 1e12 if "qkv" in gemm_ms else None,
                    "frac_of_nominal_ratio_peak": ach / int8_nominal_ratio_peak,
                    "nominal_ratio_peak": int8_nominal_ratio_peak,
                    "nominal_ratio_peak_source": f"{'4' if nv else '2'} x {peaks['source']} bf16 {regime} (timed region {region_s:.2f} s)"}
        if args.fmt in ("int4", "int4_asym", "int4_ph"):
            roofline["alu"] = {"bound": "alu", "achieved": ach_alu / 1e9, "peak": alu_peak / 1e9, "unit": "G element-steps/s",
                               "frac": ach_alu / alu_peak,
                               "note": "per-group rescale: 2 fp32 fused multiply-adds per output element and K-group; "
                                       "148 SMs x 128 fp32 lanes at the sampled SM clock"}
    kernels = {}
    for n, K, N in FLUX_SHAPES:
        t_roof = (gemm_ops[n] / int8_peak + (rot_flops[n] + 2.0 * M * RANK * N) / bf16_peak) / 1e12 * 1e3
        tot = rot_ms[n] + gemm_ms[n]
        kernels[n] = {
            "rotate_ms": rot_ms[n], "rotate_tflops": rot_flops[n] / (rot_ms[n] * 1e-3) / 1e12,
            "rotate_frac_bf16_peak": rot_flops[n] / (rot_ms[n] * 1e-3) / 1e12 / bf16_peak,
            "gemm_ms": gemm_ms[n], "gemm_tops": gemm_ops[n] / (gemm_ms[n] * 1e-3) / 1e12,
            "gemm_frac_int8_peak": gemm_ops[n] / (gemm_ms[n] * 1e-3) / 1e12 / int8_peak,
            "effective_tops": 2.0 * M * N * K / (tot * 1e-3) / 1e12,
            "frac_of_composite_roofline": t_roof / tot,
            "cublas_bf16_ms": cublas.get(n), "speedup_vs_cublas_bf16": cublas[n] / tot if n in cublas else None,
        }

    # ---- the other configurations, briefly (one GPU, headline format only): the small memory-bound layer, the PixArt
    # block linears, and the 152-linear chain of a FLUX.1-dev-shaped denoising step against the same chain in cuBLAS bf16
    configs = None
    if not args.lite and args.fmt == "int4" and world == 1 and args.configs:
        from paper_2605_16732_b200 import suite
        todo = set(args.configs.split(","))
        configs = {}
        if "1" in todo:
            configs["1"] = suite.small_m_summary(hbm_gbs=peaks["hbm_gbs"])
        if "2" in todo:
            configs["2"] = suite.pixart_block_summary()
        if "5" in todo and len(layers) == 4:
            extra = {"single_in": suite.Case(M, 3072, 21504, RANK, GROUP, synth.FLUX),
                     "single_out": suite.Case(M, 15360, 3072, RANK, GROUP, synth.FLUX)}
            run_by, cub_by, wbs = {}, {}, {}
            for L in layers:
                wbs[L["name"]] = torch.randn((L["K"], L["N"]), device=dev, dtype=torch.bfloat16) * 0.02
                run_by[L["name"]] = (lambda L=L: dq.dirotq_linear(L["x"], L["layer"], L["y"], L["ws"]))
                cub_by[L["name"]] = (lambda L=L: torch.matmul(L["x"], wbs[L["name"]]))
            for n, c in extra.items():
                run_by[n] = c.run
                cub_by[n] = (lambda c=c: torch.matmul(c.x, c.Wb))

            def all_status_zero():
                for L in layers:
                    assert dq.dirotq_workspace_status(L["ws"]) == 0
                for c in extra.values():
                    assert dq.dirotq_workspace_status(c.ws) == 0
            configs["5"] = suite.flux_step_summary(run_by, cub_by, all_status_zero, M=M)
            for c in extra.values():
                c.close()
            del wbs

    # about 10 s of CPU work: 128 token rows x 512 output columns of each of the four linears
    cpu = oracle_sample_run(1, rows=128, cols=512, fmt=args.fmt) if not args.lite else {"value": None, "unit": "TOPS", "cores": None, "kind": "oracle",
                                                      "sample": "skipped (--lite)"}
    line = {
        "metric": "dirotq_w4a4_linear_effective_tops", "value": value, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": ("nvfp4 (e2m1 x e2m1, e4m3 block scales) + bf16" if nv else "int8xint4->int32 + bf16" if args.fmt == "w4a8"
                  else "int4xint4 (exact group sums on the e4m3 tensor path) + bf16"),
        "data": "synthetic",
        "config": {"workload": WORKLOAD + _suffix(args.fmt), "M": M, "shapes": [[K, N] for _, K, N in FLUX_SHAPES], "r": RANK,
                   "group": 16 if nv else ("per-token / per-channel" if args.fmt == "w4a8" else GROUP), "format": args.fmt,
                   "l2": "inputs_exceed_l2 (each step streams > 500 MB of rotations, codes and outputs)",
                   "parallelism": f"token rows x{world}, no collective"},
        "clocks": clocks,
        "e2e": {"value": world * ops_step / (e2e_ms * 1e-3) / 1e12, "unit": "TOPS", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
        "gpu_launches": launches_per_layer * len(layers) * args.steps,
        "roofline": roofline,
        "peak_probe": peak_probe,
        "small_m": (configs or {}).get("1"),
        "configs": configs,
        "kernels": kernels,
        "frac_int8_peak_effective": value / world / int8_peak,
        # the ceiling that goes with it: the dense bf16 rotation alone caps the effective rate (per shape in `kernels`)
        "frac_of_composite_roofline": (sum(v["frac_of_composite_roofline"] * (v["rotate_ms"] + v["gemm_ms"]) for v in kernels.values())
                                       / sum(v["rotate_ms"] + v["gemm_ms"] for v in kernels.values())) if kernels else None,
        "cpu_baseline": {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")},
    }
    if not args.lite and args.fmt == "int4":
        line["cpu_baseline"]["config1_full"] = oracle_config1_full()  # a whole layer, not a sample (a fraction of a second)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--shapes", default="", help="comma-separated subset of qkv,out,mlp_up,mlp_down (profiling runs)")
    ap.add_argument("--fmt", default="int4", choices=["int4", "nvfp4", "int4_asym", "w4a8", "int4_ph", "nvfp4_ph"],
                    help="int4: the headline format (groups of 64, bf16 scales, symmetric); nvfp4: E2M1 blocks of 16 with E4M3 "
                         "scales; int4_asym: int4 with asymmetric activation codes (zero-point per group); w4a8: per-token int8 "
                         "activations, per-channel int4 weights; int4_ph: the projection form (U_h only + block-Hadamard residual), "
                         "a cheaper first stage that is not the paper's Eq. 5")
    ap.add_argument("--gemm-tile", type=int, default=0, choices=[0, 64, 66, 128, 192, 256, 512],
                    help="output columns per tile of the second kernel (int4 / int4_asym / nvfp4): 0 = chosen per call")
    ap.add_argument("--configs", default="1,2,5",
                    help="other configurations summarised in the line (int4 format, one GPU): 1 = small memory-bound layer, "
                         "2 = PixArt block linears, 5 = 152-linear FLUX step against cuBLAS bf16; empty string: none")
    ap.add_argument("--lite", action="store_true", help="skip the cuBLAS, end-to-end and CPU-baseline legs (profiling runs)")
    args = ap.parse_args()
    if args.shapes:
        keep = set(args.shapes.split(","))
        FLUX_SHAPES[:] = [t for t in FLUX_SHAPES if t[0] in keep]
    if args.impl == "reference":
        run_reference(args)
    else:
        if args.gemm_tile:
            from paper_2605_16732_b200 import binding as _dq
            _dq.dirotq_set_gemm_tile(args.gemm_tile)
        run_ours(args)


if __name__ == "__main__":
    main()
