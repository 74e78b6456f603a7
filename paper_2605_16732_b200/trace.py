"""Clock traces of the kernels' roles, read off the device.

    python -m paper_2605_16732_b200.trace [--what small_m | nvfp4 | w4a8]

Builds the diagnostic library (`build.build_trace()`: the same sources with -DDIROTQ_TRACE, in which block 0 of every kernel stamps
`clock64()` at marked points of its roles into spare 8-byte slots of the workspace's status block), runs one workload on it and
prints the stamps as cycles since the kernel's entry.  The slot map is documented at each kernel's first stamp.

    small_m   the small layer (M = 256, 1152 -> 1152, r = 32, groups of 64), each INT4 kernel replayed alone from a CUDA graph
    nvfp4     the second kernel of the NVFP4 format behind the projection form on the FLUX qkv shape (M = 4608, 3072 -> 9216)
    w4a8      the second kernel of the W4A8 format on the same shape
"""
from __future__ import annotations

import argparse
import sys


def _stamps(ws):
    import torch
    torch.cuda.synchronize()
    return ws[:256].view(torch.int64).cpu().tolist()


def _show(title, st, names, base_slot):
    base = st[base_slot]
    print(title)
    for name, slots in names:
        print("   %-58s %s" % (name, " ".join(str(st[i] - base) for i in slots)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--what", default="small_m", choices=["small_m", "nvfp4", "w4a8"])
    args = ap.parse_args()
    from . import binding as dq, build
    dq.use_library(build.build_trace())  # before the binding loads a library
    import torch  # noqa: F401  (device memory for the cases below)
    from . import suite, synth

    if args.what == "small_m":
        c = suite.Case(256, 1152, 1152, 32, 64, synth.PIXART)
        us = c.graph_ms(lambda: dq.dirotq_rotate_quantize(c.x, c.layer, c.ws)) * 1e3
        _show(f"rotate_quant_kernel (plan chosen for M = 256), {us:.2f} us per call in graph replay; cycles since entry", _stamps(c.ws),
              [("set-up done / previous grid ended", (10, 11)), ("producer: ring filled once / everything issued", (12, 13)),
               ("MMA warp: first / ninth stage seen, last tile committed", (14, 15, 16)),
               ("first epilogue warp: first accumulator seen / finished", (17, 18))], 9)
        us = c.graph_ms(lambda: dq.dirotq_w4a4_gemm(c.M, c.layer, c.ws, c.y)) * 1e3
        _show(f"w4a4_gemm_kernel (plan chosen for M = 256), {us:.2f} us per call in graph replay; cycles since entry", _stamps(c.ws),
              [("set-up done / previous grid ended", (10, 11)), ("producer: first k-block issued / everything issued", (12, 13)),
               ("first unpack warp: first stage seen / expanded", (14, 15)),
               ("MMA warp: first / fifth / last k-block, last tile committed", (16, 17, 18, 19)),
               ("first epilogue warp: first accumulator / ninth group / groups done / rank-r done / stored", (20, 21, 22, 23, 24))], 9)
        assert dq.dirotq_workspace_status(c.ws) == 0
        c.close()
        return
    suite.FMT = "nvfp4_ph" if args.what == "nvfp4" else "w4a8"
    c = suite.Case(4608, 3072, 9216, 32, 64, synth.FLUX)
    for _ in range(3):
        c.run()
    st = _stamps(c.ws)
    if args.what == "nvfp4":
        _show("nvfp4_gemm_kernel, FLUX qkv, block 0; cycles since entry (stages 6, 7, 8 of the first tile; tiles 0, 1, 2)", st,
              [("producer has issued the stage", (9, 10, 11)), ("first copier warp sees it landed", (12, 13, 14)),
               ("first / second copier warp committed", (15, 16, 17, 18, 19, 20)), ("MMA warp sees the scales ready", (21, 22, 23)),
               ("MMA warp committed the stage", (24, 25, 26)), ("epilogue tile 0: accumulator seen / released / handed over", (27, 28, 29)),
               ("epilogue tile 1", (1, 2, 3)), ("epilogue tile 2", (4, 5, 6))], 30)
    else:
        _show("w4a8_gemm_kernel, FLUX qkv, block 0; cycles since entry (stages 10, 11, 12 of the first tile; tiles 0, 1, 2)", st,
              [("producer has issued the stage", (9, 10, 11)), ("first unpack warp sees it landed", (12, 13, 14)),
               ("first unpack warp has expanded it", (15, 16, 17)), ("MMA warp starts on it", (18, 19, 20)),
               ("epilogue tile 0: accumulators seen / released / handed over", (21, 22, 23)), ("epilogue tile 1", (24, 25, 26)),
               ("epilogue tile 2", (27, 28, 29))], 30)
    assert dq.dirotq_workspace_status(c.ws) == 0
    c.close()


if __name__ == "__main__":
    sys.exit(main())
