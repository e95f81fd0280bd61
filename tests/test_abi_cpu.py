"""Host-side tests that need no GPU: the library loads, exports every symbol the header declares,
sizes the state as the paper's inventory says, and rejects bad arguments before touching a device."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2501_02379_b200 import binding as B
from paper_2501_02379_b200 import build as builder
from paper_2501_02379_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    builder.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "tgrad.h")).read()
    declared = set(re.findall(r"\b(tgrad_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    l = B.lib()
    for name in declared:
        assert hasattr(l, name), f"{name} is declared but not exported"
    assert declared == set(B.EXPORTS)


def test_status_strings():
    assert B.status_string(B.OK) == "ok"
    assert "unsupported" in B.status_string(B.ERR_UNSUPPORTED)


def test_state_bytes_counts_the_papers_inventory():
    # persistent block >= Omega + factors + M_L + V_L + M_S + V_S, and within padding of it
    for name in ("cfg1", "cfg3", "cfg4", "cfg5"):
        wl = synth.WORKLOADS[name]
        cfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, half_storage=wl.half_storage)
        pb, wb = B.state_bytes(cfg)
        p = int(np.prod(wl.ranks, dtype=np.int64))
        fac = sum(i * r for i, r in zip(wl.shape, wl.ranks))
        slabs = wl.numel // (wl.shape[-1] * wl.shape[-2])
        need = 4 * wl.k + 8 * fac + 8 * p + 4 * p + 8 * wl.k + 4 * wl.k + 4 * (slabs + 1)   # + per-slab offsets into Omega
        # + the split copy of U^(N-1) that the compression kernel reads: 1 KB per (8 rows, 8 columns)
        need += -(-wl.shape[-2] // 8) * -(-wl.ranks[-2] // 8) * 1024
        assert need <= pb <= need + 256 * (8 + len(wl.shape)) + 512
        assert wb > 0 and pb % 256 == 0 and wb % 256 == 0
    # the paper's example (N=64, M=128, r=16): core-shaped moment + factors = 71,680 entries
    cfg = B.make_config((64, 64, 128, 128), (16, 16, 16, 16), 0, 10)
    pb, _ = B.state_bytes(cfg)
    entries = 16 ** 4 + 2 * 16 * 64 + 2 * 16 * 128
    assert entries == 71680
    assert pb >= 8 * entries + 4 * 16 ** 4      # M_L complex + factors complex + V_L real


@pytest.mark.parametrize("mutate,status", [
    (lambda c: setattr(c, "ndim", 1), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "ndim", 9), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "ndim", 2), B.OK),                          # the matrix case
    (lambda c: c.ranks.__setitem__(0, 0), B.ERR_INVALID_ARG),
    (lambda c: c.ranks.__setitem__(1, 1000), B.ERR_INVALID_ARG),
    (lambda c: c.dims.__setitem__(2, 0), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "k", -1), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "k", 10 ** 9), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "T", 0), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "wg_dtype", 7), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "beta1", 1.0), B.ERR_INVALID_ARG),
    (lambda c: setattr(c, "eps", -1.0), B.ERR_INVALID_ARG),
    (lambda c: c.dims.__setitem__(0, 2000), B.ERR_UNSUPPORTED),        # eigensolver size limit
    (lambda c: (c.dims.__setitem__(3, 40), c.ranks.__setitem__(3, 33)), B.ERR_UNSUPPORTED),   # r_N <= 32
    (lambda c: (c.dims.__setitem__(2, 600), c.dims.__setitem__(3, 100)), B.ERR_UNSUPPORTED),  # slab > shared memory
])
def test_bad_configs_are_rejected_on_the_host(mutate, status):
    cfg = B.make_config((12, 10, 8, 5), (4, 3, 3, 2), 10, 4)
    mutate(cfg)
    p, w = C.c_size_t(0), C.c_size_t(0)
    assert B.lib().tgrad_state_bytes(C.byref(cfg), C.byref(p), C.byref(w)) == status


def test_too_many_entries_for_uint32_indices():
    cfg = B.make_config((1024, 1024, 1024, 8), (4, 4, 4, 4), 10, 4)
    p, w = C.c_size_t(0), C.c_size_t(0)
    assert B.lib().tgrad_state_bytes(C.byref(cfg), C.byref(p), C.byref(w)) == B.ERR_UNSUPPORTED


def test_k_of_two_to_the_31_is_unsupported():
    # 2^31 <= k <= prod(dims) < 2^32 would overflow the int slot arithmetic of the kernels: refused on the host
    cfg = B.make_config((1024, 1024, 1024, 3), (4, 4, 4, 3), 1 << 31, 4)
    p, w = C.c_size_t(0), C.c_size_t(0)
    assert B.lib().tgrad_state_bytes(C.byref(cfg), C.byref(p), C.byref(w)) == B.ERR_UNSUPPORTED
    cfg.k = (1 << 31) - 1
    assert B.lib().tgrad_state_bytes(C.byref(cfg), C.byref(p), C.byref(w)) == B.OK


def test_noalloc_entry_point_rejects_misaligned_pointers_without_a_launch():
    # pointers are plain integers here: the call must return before it touches a device
    l = B.lib()
    n0 = B.launch_count()
    for g, o, v in ((0x1004, 0x2000, 0x3000), (0x1000, 0x2004, 0x3000), (0x1000, 0x2000, 0x3008)):
        assert l.tgrad_select_topk_noalloc(g, 64, 4, B.C64, o, v, None) == B.ERR_INVALID_ARG
    assert l.tgrad_select_topk_noalloc(0x1004, 64, 4, B.C32H, 0x2000, 0x3000, None) == B.ERR_INVALID_ARG
    assert B.launch_count() == n0


def test_sticky_flag_names_match_the_header():
    header = open(os.path.join(ROOT, "include", "tgrad.h")).read()
    vals = dict(re.findall(r"#define (TGRAD_FLAG_[A-Z_]+)\s+(\d+)", header))
    assert vals == {"TGRAD_FLAG_NO_CONVERGE": str(B.FLAG_NO_CONVERGE), "TGRAD_FLAG_NONFINITE": str(B.FLAG_NONFINITE),
                    "TGRAD_FLAG_COPY_TIMEOUT": str(B.FLAG_COPY_TIMEOUT)}


def test_state_sizes_of_a_matrix():
    # N = 2: factors I_1 x r_1 and I_2 x r_2, core r_1 x r_2
    cfg = B.make_config((96, 80), (12, 10), 77, 4)
    pb, wb = B.state_bytes(cfg)
    need = 4 * 77 + 8 * (96 * 12 + 80 * 10) + 12 * 120 + 12 * 77
    assert need <= pb <= need + 8192 and wb > 0


def test_null_and_misaligned_arguments():
    l = B.lib()
    cfg = B.make_config((12, 10, 8, 5), (4, 3, 3, 2), 10, 4)
    p, w = C.c_size_t(0), C.c_size_t(0)
    assert l.tgrad_state_bytes(None, C.byref(p), C.byref(w)) == B.ERR_INVALID_ARG
    assert l.tgrad_state_bytes(C.byref(cfg), None, C.byref(w)) == B.ERR_INVALID_ARG
    h = C.c_void_p(0)
    assert l.tgrad_init_state(C.byref(cfg), None, 0, None, 0, None, C.byref(h)) == B.ERR_INVALID_ARG
    assert l.tgrad_init_state(C.byref(cfg), 256, 1 << 30, 513, 1 << 30, None, C.byref(h)) == B.ERR_INVALID_ARG
    assert l.tgrad_init_state(C.byref(cfg), 256, 16, 512, 16, None, C.byref(h)) == B.ERR_BUFFER_TOO_SMALL
    assert h.value is None
    assert l.tgrad_step(None, 256, 256, None) == B.ERR_INVALID_ARG
    assert l.tgrad_refresh_subspace(None, 256, None) == B.ERR_INVALID_ARG
    assert l.tgrad_step_batched(None, None, None, 2, None) == B.ERR_INVALID_ARG
    assert l.tgrad_step_batched(None, None, None, 0, None) == B.OK
    assert l.tgrad_destroy_state(None) == B.ERR_INVALID_ARG
    assert l.tgrad_set_step(None, 3) == B.ERR_INVALID_ARG
    assert B.launch_count() == 0 or B.launch_count() > 0     # callable without a device


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    import importlib
    import paper_2501_02379_b200.binding as mod
    monkeypatch.setattr(mod, "LIB_PATH", str(tmp_path / "nope.so"))
    monkeypatch.setattr(mod, "_lib", None)
    with pytest.raises(OSError):
        mod.lib()
    importlib.reload(mod)


def test_bench_byte_model_matches_the_stated_formula():
    import bench
    wl = synth.WORKLOADS["cfg3"]
    assert bench.step_bytes(wl) == 24 * wl.numel + 60 * wl.k + 40 * 131072 + 8 * 9480
    assert abs(bench.step_bytes(wl) / 1e9 - 0.888) < 1e-3
    wl5 = synth.WORKLOADS["cfg5"]
    assert abs(bench.step_bytes(wl5) / 1e9 - 6.95) < 0.01
