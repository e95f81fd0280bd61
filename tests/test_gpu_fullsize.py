"""Parity at the benchmark configurations' full sizes (run with -m gpu on a B200)."""
import time

import numpy as np
import pytest
import torch

from paper_2501_02379_b200 import binding as B
from paper_2501_02379_b200 import synth
from tests.parity import Pair, SampledChecker, to_device, from_device

pytestmark = pytest.mark.gpu


def test_cfg2_batched_stack_against_oracle():
    # four 64x64x32x17 tensors through the batched entry point, oracle per tensor
    wl = synth.WORKLOADS["cfg2"]
    pairs = [Pair(wl, i) for i in range(wl.n_tensors)]
    for t in range(3):
        gs_np = [p.src.gradient(t) for p in pairs]
        gs = [to_device(g, False) for g in gs_np]
        if t % wl.T == 0:
            for p, g, gd in zip(pairs, gs_np, gs):
                p.refresh(g, gd)
        B.step_batched([p.gst for p in pairs], [p.w_dev for p in pairs], gs)
        for p, g in zip(pairs, gs_np):
            from oracle import tgrad_oracle as orc
            p.w_ref = orc.oracle_step(p.ost, p.w_ref, g, refresh=False)
            p.compare()
    print("cfg2", [p.report for p in pairs][:1])


def test_cfg3_full_oracle_steps():
    wl = synth.WORKLOADS["cfg3"]
    p = Pair(wl)
    t0 = time.time()
    for t in range(2):
        p.step(t)
    print("cfg3 full oracle", p.report, f"{time.time() - t0:.1f}s")


@pytest.mark.parametrize("name", ["cfg3", "cfg4", "cfg5"])
def test_sampled_outputs_full_size(name):
    wl = synth.WORKLOADS[name]
    t0 = time.time()
    # warm-started refresh, as the benchmark runs it: the first refresh starts cold, the one forced before the
    # second step starts from the first one's eigenvectors
    c = SampledChecker(wl, n_samples=4 if name == "cfg5" else 6, warm_refresh=True)
    c.step()
    c.step(refresh=True)
    print(name, c.report, f"{time.time() - t0:.1f}s")
