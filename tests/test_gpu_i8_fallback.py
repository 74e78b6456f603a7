"""The fallback build of the library (integer tensor-core path for the W4A4 group sums, -DDIROTQ_I8_PATH).

The default build computes the integer group sums of Eq. 5 on the 8-bit float path, whose exactness is a measured
property of the part.  The fallback build computes them with int32 accumulators.  It has to stay buildable, pass the
same element-by-element parity tests against the CPU oracle, and give the same output bits as the default build.
Each build is loaded in a process of its own (the binding loads one library per process).
"""
from __future__ import annotations

import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

_DIGEST_SNIPPET = r"""
import hashlib, sys
import numpy as np, torch
sys.path.insert(0, {root!r})
from paper_2605_16732_b200 import binding as dq, synth
torch.cuda.set_device(0)
h = hashlib.sha256()
for (K, N, r, G, M, asym) in [(1152, 1152, 32, 64, 300, False), (768, 272, 128, 128, 257, False), (1152, 768, 32, 64, 130, True)]:
    spec = synth.LayerSpec(K=K, N=N, r=r, G=G, model=synth.PIXART, seed=5, calib_tokens=512)
    inp = synth.make_layer_inputs(spec, M)
    bf = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
    W, Q = torch.from_numpy(inp["W"]).cuda(), torch.from_numpy(inp["Q"]).cuda()
    prep = dq.dirotq_prepare_layer_asym if asym else dq.dirotq_prepare_layer
    layer = prep(W, Q, r, G, bias=bf(inp["bias"]))
    ws = dq.alloc_workspace(layer, M)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    dq.dirotq_linear(bf(inp["x"]), layer, y, ws)
    assert dq.dirotq_workspace_status(ws) == 0
    h.update(y.view(torch.int16).cpu().numpy().tobytes())
print("DIGEST", h.hexdigest())
"""


def _env(lib: str | None) -> dict:
    env = dict(os.environ)
    env.pop("DIROTQ_LIBRARY", None)
    if lib:
        env["DIROTQ_LIBRARY"] = lib
    return env


@pytest.fixture(scope="module")
def fallback_lib() -> str:
    from paper_2605_16732_b200 import build as _b
    return _b.build_i8()


def test_fallback_build_passes_the_parity_tests(fallback_lib):
    files = ["tests/test_gpu_parity.py", "tests/test_gpu_asym.py", "tests/test_gpu_tiles.py", "tests/test_gpu_projection_form.py"]
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider", *files],
                         cwd=ROOT, env=_env(fallback_lib), capture_output=True, text=True, timeout=1500)
    assert res.returncode == 0, res.stdout[-4000:] + res.stderr[-2000:]


def test_fallback_build_gives_the_default_build_s_bits(fallback_lib):
    digests = []
    for lib in (None, fallback_lib):
        res = subprocess.run([sys.executable, "-c", _DIGEST_SNIPPET.format(root=ROOT)], cwd=ROOT, env=_env(lib),
                             capture_output=True, text=True, timeout=600)
        assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-2000:]
        line = [ln for ln in res.stdout.splitlines() if ln.startswith("DIGEST")]
        assert line, res.stdout
        digests.append(line[0])
    assert digests[0] == digests[1]
