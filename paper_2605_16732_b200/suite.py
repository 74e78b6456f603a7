"""Timing sweep over the configurations bench.py does not time (bench.py keeps to its one-line contract).

    python -m paper_2605_16732_b200.suite [--configs 1,2,4,5] [--iters 20]

Prints one JSON line per case: both kernels' device times (CUDA events), effective TOPS
(2*M*N*K / time), the fraction of the composite roofline
t_roof = 2*M*(K-r)*N / P_int8 + (2*M*K^2 + 2*M*r*N) / P_bf16, and cuBLAS bf16 (torch.matmul) on the
same shape.  Config 5 is the chain of all 152 linears of one FLUX.1-dev-shaped denoising step,
timed device-side end to end against the same chain of bf16 GEMMs.

Run time does not depend on the rotation's values, so a seeded Householder reflection (dense,
exactly orthogonal) stands in for the PCA rotation here; activations and weights come from the
same seeded generator as everywhere else.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding as dq
from . import synth


def _peaks():
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p.get("bf16_tflops_sustained", p["bf16_tflops"]), p["hbm_gbs"], "measured"
    return 1400.0, 6650.0, "fallback"


def _bf(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _householder(K: int, seed: int) -> torch.Tensor:
    g = torch.Generator(device="cuda").manual_seed(seed)
    v = torch.randn(K, dtype=torch.float64, device="cuda", generator=g)
    v /= v.norm()
    return torch.eye(K, dtype=torch.float64, device="cuda") - 2.0 * torch.outer(v, v)


FMT = "int4"  # set from --fmt: "int4" (groups of G, bf16 scales) or "nvfp4" (blocks of 16, E4M3 scales)


class Case:
    def __init__(self, M, K, N, r, G, model):
        self.M, self.K, self.N, self.r, self.G = M, K, N, r, G
        spec = synth.LayerSpec(K=K, N=N, r=r, G=G if FMT in ("int4", "int4_asym", "int4_ph") else 64, model=model, seed=7)
        W, bias = synth.make_weights(spec)
        self.x = _bf(synth.make_tokens(spec, M, batch_seed=11))
        Wd, Q = torch.from_numpy(W).cuda(), _householder(K, K + r)
        if FMT == "nvfp4":
            # calibrate the activations' power-of-two scale on this batch through the library's own rotation
            probe = dq.dirotq_prepare_layer_nvfp4(Wd, Q, r, 0, bias=_bf(bias))
            rows = min(M, 1024)
            xrot = torch.empty((rows, K), dtype=torch.float32, device="cuda")
            dq.dirotq_rotate_quantize(self.x[:rows], probe, dq.alloc_workspace(probe, rows), xrot)
            ex = dq.dirotq_act_scale_log2_from_rotated(xrot, r)
            probe.close()
            self.layer = dq.dirotq_prepare_layer_nvfp4(Wd, Q, r, ex, bias=_bf(bias))
        elif FMT == "w4a8":
            self.layer = dq.dirotq_prepare_layer_w4a8(Wd, Q, r, bias=_bf(bias))
        elif FMT == "int4_asym":
            self.layer = dq.dirotq_prepare_layer_asym(Wd, Q, r, G, bias=_bf(bias))
        elif FMT == "int4_ph":
            self.layer = dq.dirotq_prepare_layer_ph(Wd, Q[:, :r].contiguous(), G, bias=_bf(bias))
        elif FMT == "nvfp4_ph":
            Uh = Q[:, :r].contiguous()
            self.layer = dq.dirotq_prepare_layer_nvfp4_ph(Wd, Uh, dq.dirotq_act_scale_log2_ph(self.x[:1024].contiguous(), Uh), bias=_bf(bias))
        else:
            self.layer = dq.dirotq_prepare_layer(Wd, Q, r, G, bias=_bf(bias))
        self.y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        self.ws = dq.alloc_workspace(self.layer, M)
        self.Wb = (torch.from_numpy(W).cuda()).to(torch.bfloat16)

    def run(self):
        dq.dirotq_linear(self.x, self.layer, self.y, self.ws)

    def time_kernels(self, iters):
        for _ in range(3):
            self.run()
        rot, gem = [], []
        for _ in range(iters):
            a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record()
            dq.dirotq_rotate_quantize(self.x, self.layer, self.ws)
            b.record()
            dq.dirotq_w4a4_gemm(self.M, self.layer, self.ws, self.y)
            c.record()
            torch.cuda.synchronize()
            rot.append(a.elapsed_time(b))
            gem.append(b.elapsed_time(c))
        assert dq.dirotq_workspace_status(self.ws) == 0
        cb = []
        for _ in range(3):
            torch.matmul(self.x, self.Wb)
        for _ in range(iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            torch.matmul(self.x, self.Wb)
            b.record()
            torch.cuda.synchronize()
            cb.append(a.elapsed_time(b))
        return float(np.median(rot)), float(np.median(gem)), float(np.median(cb))

    def graph_ms(self, fn, calls=10, iters=20):
        """Per-call device time of fn replayed from a CUDA graph of `calls` back-to-back calls: what a launch-bound
        small layer costs once the host is out of the way (inputs of these small shapes stay in L2 between calls)."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                fn()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(calls):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        ts = []
        for _ in range(iters):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / calls)
        return float(np.median(ts))

    def report(self, tag, iters, p_bf16, hbm, graphs=False):
        rot, gem, cb = self.time_kernels(iters)
        M, K, N, r, G = self.M, self.K, self.N, self.r, self.G
        PH, NV = FMT in ("int4_ph", "nvfp4_ph"), FMT in ("nvfp4", "nvfp4_ph")
        K_l = K if PH else K - r
        n_g = -(-K_l // G) if G else 1
        tot = rot + gem
        p_i8 = (4.0 if NV else 2.0) * p_bf16  # nominal ratio of the 4-bit / 8-bit tensor peak to bf16
        first_flops = 4.0 * M * K * max(64, -(-r // 64) * 64) if PH else 2.0 * M * K * K
        t_roof = (2.0 * M * K_l * N / p_i8 + (first_flops + 2.0 * M * r * N) / p_bf16) / 1e12 * 1e3
        if FMT == "w4a8":
            bytes_alg = 2 * M * K + 2 * K * K + K_l * N / 2 + 4 * N + 2 * 64 * N + 2 * (M * K_l * 5 + 8 * M + 2 * M * 64) + 2 * M * N
        elif NV:
            bytes_alg = 2 * M * K + 2 * K * K + K_l * N / 2 + K_l / 16 * N + 2 * 64 * N + 2 * (M * K_l / 2 + M * K_l / 16 + 2 * M * 64) + 2 * M * N
        else:
            bytes_alg = 2 * M * K + 2 * K * K + n_g * G * N / 2 + 4 * n_g * N + 2 * 64 * N + 2 * (M * n_g * G + 4 * M * n_g + 2 * M * 64) + 2 * M * N
        line = {"config": tag, "fmt": FMT, "M": M, "K": K, "N": N, "r": r, "group": G, "rotate_ms": rot, "gemm_ms": gem,
                "effective_tops": 2.0 * M * N * K / (tot * 1e-3) / 1e12,
                "frac_low_precision_peak": 2.0 * M * N * K / (tot * 1e-3) / 1e12 / p_i8,
                "frac_of_composite_roofline": t_roof / tot,
                "algorithmic_gbs": bytes_alg / (tot * 1e-3) / 1e9, "frac_hbm_peak": bytes_alg / (tot * 1e-3) / 1e9 / hbm,
                "cublas_bf16_ms": cb, "speedup_vs_cublas_bf16": cb / tot}
        if graphs:
            line["linear_graph_ms"] = self.graph_ms(self.run)
            line["cublas_bf16_graph_ms"] = self.graph_ms(lambda: torch.matmul(self.x, self.Wb))
            assert dq.dirotq_workspace_status(self.ws) == 0
        print(json.dumps(line), flush=True)

    def close(self):
        self.layer.close()


def small_m_summary(M=256, K=1152, N=1152, r=32, G=64, hbm_gbs=None):
    """The memory-bound small layer (PixArt attention projection at M = 256): device time per layer replayed from a CUDA
    graph, the bytes the method must move (activations, rotation, weight codes and scales, intermediates, output) and
    the bandwidth that amounts to."""
    c = Case(M, K, N, r, G, synth.PIXART)
    K_l = K - r
    n_g = -(-K_l // G)
    bytes_alg = 2 * M * K + 2 * K * K + n_g * G * N / 2 + 4 * n_g * N + 2 * 64 * N + 2 * (M * n_g * G + 4 * M * n_g + 2 * M * 64) + 2 * M * N
    us = c.graph_ms(c.run) * 1e3
    us_cublas = c.graph_ms(lambda: torch.matmul(c.x, c.Wb)) * 1e3
    assert dq.dirotq_workspace_status(c.ws) == 0
    c.close()
    gbs = bytes_alg / (us * 1e-6) / 1e9
    return {"workload": f"pixart_attention_projection_M{M}_K{K}_N{N}_r{r}_g{G}", "linear_graph_us": us, "cublas_bf16_graph_us": us_cublas,
            "algorithmic_bytes": bytes_alg, "algorithmic_gbs": gbs, "frac_hbm_peak": gbs / hbm_gbs if hbm_gbs else None}


def pixart_block_summary(M=4096, iters=10):
    """Config 2: the PixArt-shaped block linears at M = 4096, per shape: both kernels' device times and cuBLAS bf16."""
    out = {}
    for K, N in [(1152, 1152), (1152, 4608), (4608, 1152)]:
        c = Case(M, K, N, 32, 64, synth.PIXART)
        rot, gem, cb = c.time_kernels(iters)
        out[f"{K}x{N}"] = {"rotate_ms": rot, "gemm_ms": gem, "cublas_bf16_ms": cb, "effective_tops": 2.0 * M * N * K / ((rot + gem) * 1e-3) / 1e12}
        c.close()
    return out


def flux_step_summary(run_by_name, cublas_by_name, status_check, M=4608, reps=3):
    """Config 5: the 152 linears of one FLUX.1-dev-shaped denoising step in sequence (19 double-stream blocks of four
    linears, 38 single-stream blocks of two), device-timed, against the same chain of cuBLAS bf16 GEMMs.  `run_by_name`
    and `cublas_by_name` map a shape name to a callable that enqueues that layer once."""
    shapes = {"qkv": (3072, 9216), "out": (3072, 3072), "mlp_up": (3072, 12288), "mlp_down": (12288, 3072),
              "single_in": (3072, 21504), "single_out": (15360, 3072)}
    chain = ["qkv", "out", "mlp_up", "mlp_down"] * 19 + ["single_in", "single_out"] * 38
    res = {}
    for name, table in (("dirotq", run_by_name), ("cublas_bf16", cublas_by_name)):
        def fn():
            for n in chain:
                table[n]()
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        res[name] = float(np.median(ts))
    status_check()
    ops = sum(2.0 * M * shapes[n][0] * shapes[n][1] for n in chain)
    return {"linears": len(chain), "dirotq_chain_ms": res["dirotq"], "cublas_bf16_chain_ms": res["cublas_bf16"],
            "effective_tops": ops / (res["dirotq"] * 1e-3) / 1e12, "speedup_vs_cublas_bf16": res["cublas_bf16"] / res["dirotq"],
            "note": "one prepared layer per distinct shape is reused for every block of that shape"}


def memory_report():
    """Bytes of a prepared layer (`dirotq_layer_bytes*`, no GPU needed) against its bf16 weights, for the layer shapes of
    the configurations, at the benchmark's rank and at about a tenth of K."""
    shapes = {"pixart qkv/o": (1152, 1152), "pixart fc1": (1152, 4608), "pixart fc2": (4608, 1152),
              "flux qkv": (3072, 9216), "flux out": (3072, 3072), "flux mlp_up": (3072, 12288), "flux mlp_down": (12288, 3072),
              "flux single_in": (3072, 21504), "flux single_out": (15360, 3072)}
    for name, (K, N) in shapes.items():
        for r in (32, int(round(0.1 * K / 16)) * 16):
            full = dq.dirotq_layer_bytes(K, N, r, 64)
            sib = dq.dirotq_layer_bytes_sibling(K, N, r, 64)
            print(json.dumps({"layer": name, "K": K, "N": N, "r": r, "group": 64, "bf16_weight_bytes": 2 * K * N,
                              "layer_bytes": full, "layer_bytes_without_rotation": sib,
                              "x_smaller_than_bf16": 2.0 * K * N / full,
                              "x_smaller_than_bf16_without_rotation": 2.0 * K * N / sib}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--memory", action="store_true", help="print the layer sizes (no GPU needed) and exit")
    ap.add_argument("--configs", default="1,2,4,5", help="comma-separated subset of 1,2,3p,4,5")
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--fmt", default="int4", choices=["int4", "nvfp4", "int4_asym", "w4a8", "int4_ph", "nvfp4_ph"])
    ap.add_argument("--ranks", default="16,32,64,128", help="ranks swept by config 4")
    args = ap.parse_args()
    if args.memory:
        memory_report()
        return
    global FMT
    FMT = args.fmt
    todo = set(args.configs.split(","))
    p_bf16, hbm, src = _peaks()
    print(json.dumps({"peaks": {"bf16_tflops_sustained": p_bf16, "int8_tops": 2 * p_bf16, "fp4_tflops_nominal_ratio": 4 * p_bf16, "fmt": FMT, "hbm_gbs": hbm, "source": src}}), flush=True)

    if "1" in todo:
        c = Case(256, 1152, 1152, 32, 64, synth.PIXART)
        c.report("1: PixArt attention projection, M=256", args.iters, p_bf16, hbm, graphs=True)
        c.close()
    if "2" in todo:
        for K, N in [(1152, 1152), (1152, 4608), (4608, 1152)]:
            c = Case(4096, K, N, 32, 64, synth.PIXART)
            c.report("2: PixArt block linear, M=4096", args.iters, p_bf16, hbm, graphs=True)
            c.close()
    if "2" in todo and FMT == "int4":
        # q, k, v of a PixArt block read the same activations: one rotate/quantize pass, three second-kernel launches
        cs = [Case(4096, 1152, 1152, 32, 64, synth.PIXART) for _ in range(3)]
        def shared():
            dq.dirotq_rotate_quantize(cs[0].x, cs[0].layer, cs[0].ws)
            for c in cs:
                dq.dirotq_w4a4_gemm(c.M, c.layer, cs[0].ws, c.y)
        def separate():
            for c in cs:
                dq.dirotq_linear(cs[0].x, c.layer, c.y, c.ws)
        res = {}
        for name, fn in (("shared_rotation", shared), ("separate", separate)):
            for _ in range(3):
                fn()
            ts = []
            for _ in range(args.iters):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            res[name] = float(np.median(ts))
        print(json.dumps({"config": "2: PixArt q/k/v projections (3 x 1152 -> 1152, M=4096) on one shared rotation",
                          "shared_rotation_ms": res["shared_rotation"], "separate_ms": res["separate"],
                          "speedup": res["separate"] / res["shared_rotation"]}), flush=True)
        for c in cs:
            c.close()
    if "3p" in todo:
        # the FLUX linears at the paper's own rank, about a tenth of K kept in 16 bits (Sec. 4.2), instead of r = 32
        for K, N, r in [(3072, 9216, 320), (3072, 3072, 320), (3072, 12288, 320), (12288, 3072, 1232)]:
            c = Case(4608, K, N, r, 64, synth.FLUX)
            c.report("3p: FLUX linear, M=4608, r = 10 % of K", args.iters, p_bf16, hbm)
            c.close()
    if "4" in todo:
        for K, N in [(3072, 9216), (12288, 3072)]:
            for r in [int(v) for v in args.ranks.split(",")]:
                for G in ((64, 128) if FMT in ("int4", "int4_asym", "int4_ph") else (16,) if FMT in ("nvfp4", "nvfp4_ph") else (0,)):
                    c = Case(18432, K, N, r, G, synth.FLUX)
                    c.report("4: FLUX batch 4 (M=18432) rank/group sweep", max(5, args.iters // 2), p_bf16, hbm)
                    c.close()
                    torch.cuda.empty_cache()
    if "5" in todo:
        M = 4608
        shapes = {"qkv": (3072, 9216), "out": (3072, 3072), "mlp_up": (3072, 12288), "mlp_down": (12288, 3072),
                  "single_in": (3072, 21504), "single_out": (15360, 3072)}
        cases = {n: Case(M, K, N, 32, 64, synth.FLUX) for n, (K, N) in shapes.items()}
        # 19 double-stream blocks (4 linears, both streams as one M = 4608 batch) + 38 single-stream blocks (2 linears)
        chain = ["qkv", "out", "mlp_up", "mlp_down"] * 19 + ["single_in", "single_out"] * 38
        assert len(chain) == 152

        def run_ours():
            for n in chain:
                cases[n].run()

        def run_cublas():
            for n in chain:
                torch.matmul(cases[n].x, cases[n].Wb)

        res = {}
        for name, fn in (("dirotq", run_ours), ("cublas_bf16", run_cublas)):
            fn()
            torch.cuda.synchronize()
            ts = []
            for _ in range(5):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            res[name] = float(np.median(ts))
        for c in cases.values():
            assert dq.dirotq_workspace_status(c.ws) == 0
        ops = sum(2.0 * M * shapes[n][0] * shapes[n][1] for n in chain)
        print(json.dumps({"config": "5: one FLUX.1-dev-shaped denoising step, 152 linears, M=4608",
                          "note": "one prepared layer per distinct shape is reused for every block of that shape",
                          "dirotq_chain_ms": res["dirotq"], "cublas_bf16_chain_ms": res["cublas_bf16"],
                          "effective_tops": ops / (res["dirotq"] * 1e-3) / 1e12,
                          "speedup_vs_cublas_bf16": res["cublas_bf16"] / res["dirotq"]}), flush=True)


if __name__ == "__main__":
    main()
