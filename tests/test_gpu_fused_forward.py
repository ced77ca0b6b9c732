"""The one-kernel form of a layer's forward pass (Eqs. 2-3: aggregation rows built in shared memory as the A operand of the
dense transform, E2EGREC_FUSED_FORWARD=1) against the oracle and against the default two-kernel path."""
import os
import subprocess
import sys

import numpy as np
import pytest

from fused_forward_case import make_case
from test_gpu_parity import _check_float

pytestmark = pytest.mark.gpu
HERE = os.path.dirname(os.path.abspath(__file__))


def _run_child(name, path, fused):
    env = dict(os.environ)
    env.pop("E2EGREC_FUSED_FORWARD", None)
    if fused:
        env["E2EGREC_FUSED_FORWARD"] = "1"
    env["PYTHONPATH"] = os.pathsep.join([os.path.dirname(HERE), HERE, env.get("PYTHONPATH", "")])
    subprocess.run([sys.executable, os.path.join(HERE, "fused_forward_case.py"), name, path], env=env, check=True, timeout=600)
    return dict(np.load(path))


@pytest.mark.parametrize("name", ["d128", "d256_three_layers", "d64_take_all"])
def test_fused_layer_matches_oracle_and_the_two_kernel_bits(name, tmp_path):
    fused = _run_child(name, str(tmp_path / "fused.npz"), True)
    plain = _run_child(name, str(tmp_path / "plain.npz"), False)
    n_layers = len([k for k in fused if k.startswith("dW")])
    # one launch per layer instead of two: the fused kernel did run
    assert int(plain["launches"][0]) - int(fused["launches"][0]) == n_layers
    # same sums in the same order, same rounding points: identical bits everywhere downstream
    for k in plain:
        if k != "launches":
            assert np.array_equal(fused[k], plain[k]), k
    # and the oracle, element by element
    case = make_case(name)
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    ora = case.run_oracle(dH)
    gpu = dict(out=fused["out"], dX=fused["dX"], dWs=[fused[f"dW{l}"] for l in range(n_layers)],
               layer_out=[fused[f"h{l}"] for l in range(n_layers)])
    _check_float(case, gpu, ora)
