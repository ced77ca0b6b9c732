"""Run by tests/test_gpu_fused_forward.py in a child process (the library reads E2EGREC_FUSED_FORWARD once per process):
forward + backward of one seeded case on the GPU, results written to the .npz file named on the command line."""
import dataclasses
import sys

import numpy as np

import synth_inputs as S
from helpers import Case


def make_case(name):
    base = S.WORKLOADS["medium_small"]
    if name == "d128":
        return Case(base, step=1)
    if name == "d256_three_layers":
        return Case(dataclasses.replace(base, dim=256, hidden=256, fanouts=(6, 4, 3), batch=700), step=2)
    if name == "d64_take_all":       # fanout above most degrees: rows with fewer neighbours than the fanout, and none
        return Case(dataclasses.replace(base, dim=64, hidden=96, fanouts=(40,), batch=333), step=3)
    raise ValueError(name)


def main(name, path):
    import paper_2511_20564_b200 as E
    case = make_case(name)
    dH = case.upstream_grad(case.seeds.size, case.w.hidden)
    before = E.launch_count()
    gpu = case.run_gpu(dH)
    arrays = dict(out=gpu["out"], dX=gpu["dX"], launches=np.array([E.launch_count() - before]))
    for l, a in enumerate(gpu["dWs"]):
        arrays[f"dW{l}"] = a
    for l, a in enumerate(gpu["layer_out"]):
        arrays[f"h{l}"] = a
    np.savez(path, **arrays)


if __name__ == "__main__":
    main(sys.argv[1], sys.argv[2])
