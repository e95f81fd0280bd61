"""The allocation-free top-k entry point against the regular refresh and the CPU oracle (run with -m gpu on a B200).

Some callers of this library may not allocate device memory while they call it: an allocator
hook that would re-enter itself, a process whose device memory was handed out in full at
start-up.  tgrad_select_topk_noalloc serves them with scratch built into the library.  Here it
must give, twice in a row on different inputs (the scratch keeps the first call's leftovers),
exactly the index set the regular refresh stores, and the values of the gradient there.
This file is collected last on purpose, so a run that stops at the first failure has already
run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import tgrad_oracle as orc
from paper_2501_02379_b200 import binding as B
from paper_2501_02379_b200 import synth
from tests.parity import to_device

pytestmark = pytest.mark.gpu


def _reference_omega(g_dev, shape, ranks, k):
    st = B.TgradState(B.make_config(shape, ranks, k, 4, auto_refresh=False))
    st.refresh_subspace(g_dev)
    return st.export(B.WHAT_OMEGA)


def test_noalloc_topk_matches_refresh_twice_in_a_row():
    wl = synth.WORKLOADS["ragged4"]
    src = synth.GradientSource(wl)
    cases = [(src.gradient(0), wl.k), (synth.quantised_ties(wl.shape, 5, 3).astype(np.complex64), 3 * wl.k + 1)]
    omega = torch.empty(max(k for _, k in cases), dtype=torch.int32, device="cuda")      # bit pattern of uint32
    values = torch.empty(max(k for _, k in cases), 2, dtype=torch.float32, device="cuda")
    for g, k in cases:
        g_dev = to_device(g, False)
        omega.fill_(-1); values.fill_(float("nan"))
        B.select_topk_noalloc(g_dev, g.size, k, omega, values)
        torch.cuda.synchronize()
        got = omega[:k].cpu().numpy().view(np.uint32)
        want = _reference_omega(g_dev, wl.shape, wl.ranks, k)
        assert np.array_equal(got, want)                                   # integer work: bit-exact
        assert np.array_equal(got, orc.sparse_indices_topk(g, k))          # and what the definition gives
        vals = values[:k].cpu().numpy().view(np.complex64)[:, 0]
        assert np.array_equal(vals, g.reshape(-1)[want.astype(np.int64)])  # a gather: bit-exact


def test_noalloc_rejects_oversized_and_bad_arguments():
    g = torch.zeros(16, 2, dtype=torch.float32, device="cuda")
    o = torch.zeros(4, dtype=torch.int32, device="cuda")
    v = torch.zeros(4, 2, dtype=torch.float32, device="cuda")
    with pytest.raises(B.TgradError) as e:
        B.select_topk_noalloc(g, B.NOALLOC_MAX_NUMEL + 1, 4, o, v)
    assert e.value.status == B.ERR_TOO_LARGE and "scratch" in str(e.value)
    with pytest.raises(B.TgradError) as e:
        B.select_topk_noalloc(g, 16, 17, o, v)
    assert e.value.status == B.ERR_INVALID_ARG
