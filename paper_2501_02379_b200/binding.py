"""Thin ctypes binding of the C ABI in include/tgrad.h.

Argument marshalling only: every step of the optimizer runs in the CUDA
library.  PyTorch is used to own device memory and streams.  If the library
is missing, loading raises -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtgrad.so")
MAX_NDIM = 8
NUM_STAGES = 5
STAGE_NAMES = ["proj_tail", "proj_chain", "mode1_adam", "back_chain", "back_tail"]

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_BUFFER_TOO_SMALL, ERR_CUDA, ERR_NO_CONVERGE, ERR_NONFINITE, ERR_BAD_STATE = range(8)
ERR_TOO_LARGE = 8
NOALLOC_MAX_NUMEL = 1 << 26
FLAG_NO_CONVERGE, FLAG_NONFINITE, FLAG_COPY_TIMEOUT = 1, 2, 4
C64, C32H, C32B = 0, 1, 2
COMPOSITIONS = {"us_lr": 0, "lr_us": 1, "sum": 2}
STRATEGIES = {"topk": 0, "randk": 1, "probk": 2}
WHAT_OMEGA, WHAT_M_L, WHAT_V_L, WHAT_M_S, WHAT_V_S, WHAT_CORE, WHAT_N_L, WHAT_N_S = 1, 2, 3, 4, 5, 6, 7, 8
WHAT_GRAM_BASE, WHAT_FACTOR_BASE = 32, 64


class TgradConfig(C.Structure):
    _fields_ = [
        ("ndim", C.c_int32),
        ("dims", C.c_int64 * MAX_NDIM),
        ("ranks", C.c_int32 * MAX_NDIM),
        ("k", C.c_int64),
        ("T", C.c_int32),
        ("lr", C.c_float), ("alpha", C.c_float), ("lambda_", C.c_float),
        ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("weight_decay", C.c_float),
        ("wg_dtype", C.c_int32),
        ("auto_refresh", C.c_int32),
        ("jacobi_max_sweeps", C.c_int32),
        ("jacobi_tol", C.c_float),
        ("warm_refresh", C.c_int32),
        ("hooi_iters", C.c_int32),
        ("composition", C.c_int32),
        ("sparse_strategy", C.c_int32),
        ("seed", C.c_uint64),
    ]


class TgradError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None

EXPORTS = [
    "tgrad_state_bytes", "tgrad_init_state", "tgrad_step", "tgrad_refresh_subspace", "tgrad_step_batched",
    "tgrad_refresh_subspace_batched", "tgrad_query_status", "tgrad_export_state", "tgrad_import_state",
    "tgrad_set_step", "tgrad_destroy_state", "tgrad_status_string", "tgrad_launch_count",
    "tgrad_set_stage_timing", "tgrad_get_stage_times", "tgrad_select_topk_noalloc", "tgrad_diagnostics",
]


def lib() -> C.CDLL:
    """Load libtgrad.so (once).  Raises OSError if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError(f"{LIB_PATH} is missing: build it with paper_2501_02379_b200.build.build() "
                          "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        vp, sz = C.c_void_p, C.c_size_t
        cfgp = C.POINTER(TgradConfig)
        l.tgrad_state_bytes.argtypes = [cfgp, C.POINTER(sz), C.POINTER(sz)]
        l.tgrad_init_state.argtypes = [cfgp, vp, sz, vp, sz, vp, C.POINTER(vp)]
        l.tgrad_step.argtypes = [vp, vp, vp, vp]
        l.tgrad_refresh_subspace.argtypes = [vp, vp, vp]
        l.tgrad_step_batched.argtypes = [C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.c_int32, vp]
        l.tgrad_refresh_subspace_batched.argtypes = [C.POINTER(vp), C.POINTER(vp), C.c_int32, vp]
        l.tgrad_query_status.argtypes = [vp, vp, C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_int32)]
        l.tgrad_export_state.argtypes = [vp, C.c_int32, vp, sz, vp]
        l.tgrad_import_state.argtypes = [vp, C.c_int32, vp, sz, vp]
        l.tgrad_set_step.argtypes = [vp, C.c_int64]
        l.tgrad_destroy_state.argtypes = [vp]
        l.tgrad_status_string.argtypes = [C.c_int]
        l.tgrad_status_string.restype = C.c_char_p
        l.tgrad_launch_count.argtypes = []
        l.tgrad_launch_count.restype = C.c_int64
        l.tgrad_set_stage_timing.argtypes = [vp, C.c_int32]
        l.tgrad_get_stage_times.argtypes = [vp, vp, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        l.tgrad_select_topk_noalloc.argtypes = [vp, C.c_int64, C.c_int64, C.c_int32, vp, vp, vp]
        l.tgrad_diagnostics.argtypes = [vp, vp, vp, C.POINTER(C.c_double)]
        for name in EXPORTS:
            if name not in ("tgrad_status_string", "tgrad_launch_count"):
                getattr(l, name).restype = C.c_int
        _lib = l
    return _lib


def status_string(s: int) -> str:
    return lib().tgrad_status_string(int(s)).decode()


def launch_count() -> int:
    return int(lib().tgrad_launch_count())


def _check(s: int, where: str) -> None:
    if s != OK:
        raise TgradError(s, where)


def make_config(shape: Sequence[int], ranks: Sequence[int], k: int, T: int, lr: float = 1e-3, alpha: float = 1.0,
                lam: float = 1.0, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                weight_decay: float = 0.0, half_storage: bool = False, bf16_storage: bool = False, auto_refresh: bool = True,
                jacobi_max_sweeps: int = 0, jacobi_tol: float = 0.0, warm_refresh: bool = False,
                hooi_iters: int = 0, composition: str = "us_lr", strategy: str = "topk", seed: int = 0) -> TgradConfig:
    if len(shape) > MAX_NDIM or len(shape) != len(ranks):
        raise ValueError("bad shape / ranks")
    cfg = TgradConfig()
    cfg.ndim = len(shape)
    for i, (d, r) in enumerate(zip(shape, ranks)):
        cfg.dims[i] = int(d)
        cfg.ranks[i] = int(r)
    cfg.k = int(k)
    cfg.T = int(T)
    cfg.lr, cfg.alpha, cfg.lambda_ = lr, alpha, lam
    cfg.beta1, cfg.beta2, cfg.eps = beta1, beta2, eps
    cfg.weight_decay = weight_decay
    cfg.wg_dtype = C32B if bf16_storage else (C32H if half_storage else C64)
    cfg.auto_refresh = 1 if auto_refresh else 0
    cfg.jacobi_max_sweeps = jacobi_max_sweeps
    cfg.jacobi_tol = jacobi_tol
    cfg.warm_refresh = 1 if warm_refresh else 0
    cfg.hooi_iters = int(hooi_iters)
    cfg.composition = COMPOSITIONS[composition]
    cfg.sparse_strategy = STRATEGIES[strategy]
    cfg.seed = int(seed)
    return cfg


def state_bytes(cfg: TgradConfig):
    p, w = C.c_size_t(0), C.c_size_t(0)
    _check(lib().tgrad_state_bytes(C.byref(cfg), C.byref(p), C.byref(w)), "tgrad_state_bytes")
    return int(p.value), int(w.value)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if hasattr(stream, "cuda_stream"):
        return stream.cuda_stream
    return int(stream)


class TgradState:
    """One optimizer state (one weight tensor).  Device blocks are torch uint8
    tensors owned by this object; the library only borrows them."""

    def __init__(self, cfg: TgradConfig, device="cuda", stream=None):
        import torch
        self.cfg = cfg
        self.shape = tuple(int(cfg.dims[i]) for i in range(cfg.ndim))
        self.ranks = tuple(int(cfg.ranks[i]) for i in range(cfg.ndim))
        self.k = int(cfg.k)
        self.core_entries = int(np.prod(self.ranks, dtype=np.int64))
        pb, wb = state_bytes(cfg)
        self.persistent = torch.empty(max(pb, 256), dtype=torch.uint8, device=device)
        self.workspace = torch.empty(max(wb, 256), dtype=torch.uint8, device=device)
        h = C.c_void_p(0)
        _check(lib().tgrad_init_state(C.byref(cfg), self.persistent.data_ptr(), pb, self.workspace.data_ptr(), wb,
                                      _stream_ptr(stream), C.byref(h)), "tgrad_init_state")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            lib().tgrad_destroy_state(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # --- the hot path -------------------------------------------------------------
    def step(self, weight, grad, stream=None):
        _check(lib().tgrad_step(self.handle, weight.data_ptr(), grad.data_ptr(), _stream_ptr(stream)), "tgrad_step")

    def refresh_subspace(self, grad, stream=None):
        _check(lib().tgrad_refresh_subspace(self.handle, grad.data_ptr(), _stream_ptr(stream)),
               "tgrad_refresh_subspace")

    # --- status / inspection ---------------------------------------------------------
    def query_status(self, stream=None):
        flags, t = C.c_int32(0), C.c_int64(0)
        sweeps = (C.c_int32 * MAX_NDIM)()
        _check(lib().tgrad_query_status(self.handle, _stream_ptr(stream), C.byref(flags), C.byref(t), sweeps),
               "tgrad_query_status")
        return int(flags.value), int(t.value), [int(sweeps[i]) for i in range(self.cfg.ndim)]

    def _spec(self, what):
        k, p = self.k, self.core_entries
        if what == WHAT_OMEGA:
            return (k,), np.uint32
        if what in (WHAT_M_L, WHAT_CORE, WHAT_N_L):
            return self.ranks, np.complex64
        if what == WHAT_V_L:
            return self.ranks, np.float32
        if what in (WHAT_M_S, WHAT_N_S):
            return (k,), np.complex64
        if what == WHAT_V_S:
            return (k,), np.float32
        if WHAT_FACTOR_BASE <= what < WHAT_FACTOR_BASE + self.cfg.ndim:
            n = what - WHAT_FACTOR_BASE
            return (self.shape[n], self.ranks[n]), np.complex64
        if WHAT_GRAM_BASE <= what < WHAT_GRAM_BASE + self.cfg.ndim:
            n = what - WHAT_GRAM_BASE
            return (self.shape[n], self.shape[n]), np.complex64
        raise ValueError(what)

    def export(self, what, stream=None) -> np.ndarray:
        shape, dt = self._spec(what)
        out = np.empty(shape, dtype=dt)
        _check(lib().tgrad_export_state(self.handle, what, out.ctypes.data, out.nbytes, _stream_ptr(stream)),
               "tgrad_export_state")
        return out

    def import_(self, what, arr: np.ndarray, stream=None):
        shape, dt = self._spec(what)
        a = np.ascontiguousarray(arr, dtype=dt)
        if a.shape != tuple(shape):
            raise ValueError("shape mismatch")
        _check(lib().tgrad_import_state(self.handle, what, a.ctypes.data, a.nbytes, _stream_ptr(stream)),
               "tgrad_import_state")

    def factors(self) -> List[np.ndarray]:
        return [self.export(WHAT_FACTOR_BASE + n) for n in range(self.cfg.ndim)]

    def set_step(self, t: int):
        _check(lib().tgrad_set_step(self.handle, int(t)), "tgrad_set_step")

    def diagnostics(self, grad, stream=None):
        """(||G||_F, sparse share, low-rank reconstruction error relative to ||G||_F, orthonormality defect) of the last step."""
        out = (C.c_double * 4)()
        _check(lib().tgrad_diagnostics(self.handle, grad.data_ptr(), _stream_ptr(stream), out), "tgrad_diagnostics")
        return tuple(float(out[i]) for i in range(4))

    def set_stage_timing(self, on: bool):
        _check(lib().tgrad_set_stage_timing(self.handle, 1 if on else 0), "tgrad_set_stage_timing")

    def stage_times(self, stream=None):
        ms = (C.c_float * NUM_STAGES)()
        n = C.c_int32(0)
        _check(lib().tgrad_get_stage_times(self.handle, _stream_ptr(stream), ms, C.byref(n)), "tgrad_get_stage_times")
        return [float(ms[i]) for i in range(NUM_STAGES)], int(n.value)


def step_batched(states: Sequence[TgradState], weights, grads, stream=None):
    n = len(states)
    hs = (C.c_void_p * n)(*[s.handle for s in states])
    ws = (C.c_void_p * n)(*[w.data_ptr() for w in weights])
    gs = (C.c_void_p * n)(*[g.data_ptr() for g in grads])
    _check(lib().tgrad_step_batched(hs, ws, gs, n, _stream_ptr(stream)), "tgrad_step_batched")


def refresh_subspace_batched(states: Sequence[TgradState], grads, stream=None):
    n = len(states)
    hs = (C.c_void_p * n)(*[s.handle for s in states])
    gs = (C.c_void_p * n)(*[g.data_ptr() for g in grads])
    _check(lib().tgrad_refresh_subspace_batched(hs, gs, n, _stream_ptr(stream)), "tgrad_refresh_subspace_batched")


def select_topk_noalloc(grad, numel: int, k: int, omega_out, values_out, half_storage: bool = False, stream=None):
    """Top-k index set and values of `grad` through the entry point that allocates nothing:
    its scratch is a fixed array inside the library, so it serves callers that must not call
    cudaMalloc (allocator hooks, fully pre-partitioned device memory).  `omega_out` (k x uint32)
    and `values_out` (k x complex64 as float pairs) are device tensors the caller already owns.
    Calls share that scratch: keep them on one stream."""
    _check(lib().tgrad_select_topk_noalloc(grad.data_ptr(), int(numel), int(k), C32H if half_storage else C64,
                                           omega_out.data_ptr() if k else None, values_out.data_ptr() if k else None,
                                           _stream_ptr(stream)), "tgrad_select_topk_noalloc")
