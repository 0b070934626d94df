"""PD_LOG=1 makes every launcher name the kernel variant it chose, one line per launch on stderr; without it
nothing is printed.  Run in child processes because the variable is read once per process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import torch
from paper_2511_03586_b200 import api
x = torch.randn(64, 512, device="cuda")
api.pd_softmax(x)
api.pd_layernorm(torch.randn(8, 4096, device="cuda"), torch.ones(4096, device="cuda"), torch.zeros(4096, device="cuda"), 1e-5)
a = torch.randn(512, 256, device="cuda").to(torch.bfloat16)
b = torch.randn(256, 512, device="cuda").to(torch.bfloat16)
api.pd_gemm_bf16(a, b)
api.pd_attention_fwd(torch.randn(128, 192, device="cuda").to(torch.bfloat16), batch=1, seq=128, heads=1)
torch.cuda.synchronize()
"""


def _run(env_value):
    env = dict(os.environ, PYTHONPATH=ROOT)
    env.pop("PD_LOG", None)
    if env_value is not None:
        env["PD_LOG"] = env_value
    r = subprocess.run([sys.executable, "-c", SCRIPT], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    return [line for line in r.stderr.splitlines() if line.startswith("pd: ")]


def test_variant_selection_is_logged_on_request():
    lines = _run("1")
    assert any(l.startswith("pd: softmax 64 x 512: one warp per row") for l in lines), lines
    assert any(l.startswith("pd: layernorm 8 x 4096: one CTA per row") for l in lines), lines
    assert any(l.startswith("pd: gemm 512 x 512 x 256") and "tiles" in l for l in lines), lines
    assert any(l.startswith("pd: attention batch 1 seq 128 heads 1: fused kernel") for l in lines), lines
    assert _run(None) == []
    assert _run("0") == []
