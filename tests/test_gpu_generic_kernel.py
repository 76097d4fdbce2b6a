"""The tensor-core kernel exists in two forms: specialised on (row-norm, activation), which serves
every call, and generic (both read at run time), which runs when a switch of the kernel is set.  Switch 128 selects plain register stores instead of staged TMA stores
and leaves the results right, so a child process run with it drives the generic form -- and the
other store path -- over the same shapes; its outputs must equal the specialised form's bit for bit.
Runs in a child process because the switches are read once per process."""
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2603_12440_b200 import inputs

ROOT = Path(__file__).resolve().parent.parent

CASES = [  # M, N, K, act, norm, bias, residual
    (300, 520, 200, "gelu_erf", "layernorm", True, True),
    (257, 1032, 136, "silu", "softmax", False, True),
    (515, 264, 72, "relu", "rmsnorm", True, False),
    (260, 2056, 64, "sigmoid", "none", True, True),
    (100, 1032, 200, "gelu_tanh", "softmax", True, False),      # one row block: single CTAs instead of pairs
]

CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
import paper_2603_12440_b200 as kf
from tests.test_gpu_generic_kernel import CASES, outputs
np.savez(sys.argv[1], *[o.view(torch.int16).cpu().numpy() for o in outputs(kf)])
"""


def outputs(kf):
    outs = []
    for i, (M, N, K, act, norm, bias, res) in enumerate(CASES):
        p = inputs.make_problem(f"g{i}", "bf16", M, N, K, seed=500 + i, std_x=1.0, std_w=1.0 / np.sqrt(K),
                                bias_std=0.5 if bias else None, residual_std=1.0 if res else None,
                                gamma_std=0.1 if norm in ("layernorm", "rmsnorm") else None,
                                beta_std=0.1 if norm == "layernorm" else None, act=act, norm=norm)
        d = inputs.problem_to_torch(p)
        assert kf.tile_config(M, N, K, torch.bfloat16, norm)["cta_group"] == (2 if M > 128 else 1)
        outs.append(kf.linear_epilogue_rownorm(d["X"], d["W"], d["bias"], p.act, p.scale, d["residual"], p.norm,
                                               d["gamma"], d["beta"], p.eps))
    kf.check_device_status()
    return outs


@pytest.mark.gpu
def test_generic_form_with_register_stores_equals_the_specialised_form(tmp_path):
    import paper_2603_12440_b200 as kf
    if os.environ.get("KF_TC_DEBUG"):
        pytest.skip("this process already runs with a kernel switch set")
    want = outputs(kf)
    f = tmp_path / "generic.npz"
    env = dict(os.environ, KF_TC_DEBUG="128")
    out = subprocess.run([sys.executable, "-c", CHILD % str(ROOT), str(f)], env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    got = np.load(f)
    for i, w in enumerate(want):
        assert np.array_equal(got[f"arr_{i}"], w.view(torch.int16).cpu().numpy()), f"case {i}: {CASES[i]}"
