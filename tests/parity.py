"""Harness that runs the CUDA library and the CPU oracle side by side.

Protocol: Omega is compared bit-exactly at every refresh; the refreshed U^(n)
are compared as subspaces (principal angles) and then the GPU's factors are
copied into the oracle ("U-sync"), because Adam's element-wise normalisation
depends on the basis chosen inside the subspace, which eigenvectors fix only up
to phases and rotations of (nearly) degenerate eigenspaces.  Everything
downstream is then compared element-wise under identical factors.
"""
import numpy as np
import torch

from oracle import tgrad_oracle as orc
from paper_2501_02379_b200 import binding as B
from paper_2501_02379_b200 import synth
from tests import helpers as H

TOL_FLOAT = 1e-4       # max relative error, entries measured against max(|ref|, 1e-3 rms(ref))
TOL_ANGLE = 1e-3       # largest principal-angle sine of a refreshed factor
TOL_ORTHO = 1e-5       # max |U^H U - I|


def to_device(x: np.ndarray, half: bool) -> torch.Tensor:
    """complex64 array -> device tensor in the storage layout (float32 or float16 pairs)."""
    if half:
        return torch.from_numpy(synth.to_half_pairs(x)).cuda()
    return torch.from_numpy(np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,))).cuda()


def from_device(t: torch.Tensor, half: bool) -> np.ndarray:
    a = t.cpu().numpy()
    if half:
        return synth.from_half_pairs(a)
    return np.ascontiguousarray(a).view(np.complex64)[..., 0]


def storage_exact(x: np.ndarray, half: bool) -> np.ndarray:
    return synth.from_half_pairs(synth.to_half_pairs(x)) if half else x


class Pair:
    def __init__(self, wl: synth.Workload, tensor_id=0, **over):
        self.wl = wl
        self.src = synth.GradientSource(wl, tensor_id)
        kw = dict(lr=wl.lr, alpha=1.0, lam=1.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
        kw.update(over)
        self.half = wl.half_storage
        self.ocfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, half_storage=self.half, **kw)
        self.ost = orc.OracleState(self.ocfg)
        self.gcfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, half_storage=self.half, auto_refresh=False, **kw)
        self.gst = B.TgradState(self.gcfg)
        w0 = storage_exact(self.src.weight(), self.half)
        self.w_ref = w0
        self.w_dev = to_device(w0, self.half)
        self.report = {}

    def _note(self, name, val):
        self.report[name] = max(self.report.get(name, 0.0), float(val))

    def refresh(self, g: np.ndarray, g_dev: torch.Tensor):
        before = g_dev.clone()
        self.gst.refresh_subspace(g_dev)
        flags, _, sweeps = self.gst.query_status()
        assert flags == 0, f"sticky flags {flags}, sweeps {sweeps}"
        assert torch.equal(before, g_dev), "refresh must leave the gradient as it found it"
        orc.oracle_refresh(self.ost, g)
        om = self.gst.export(B.WHAT_OMEGA)
        assert np.array_equal(om, self.ost.omega), "Omega differs from the oracle"
        us = self.gst.factors()
        for n, (ug, uo) in enumerate(zip(us, self.ost.factors)):
            ang = H.max_sin_angle(ug, uo)
            self._note("angle", ang)
            assert ang <= TOL_ANGLE, f"mode {n}: principal angle sine {ang}"
            od = H.ortho_defect(ug)
            self._note("ortho", od)
            assert od <= TOL_ORTHO, f"mode {n}: orthonormality defect {od}"
            # canonical phase: largest-modulus component of each column is real positive
            for j in range(ug.shape[1]):
                i = int(np.argmax(np.abs(ug[:, j])))
                assert abs(ug[i, j].imag) <= 1e-6 * abs(ug[i, j]) + 1e-12 and ug[i, j].real > 0
        self.ost.factors = [u.copy() for u in us]       # U-sync
        return sweeps

    def step(self, t: int, check=True):
        g = storage_exact(self.src.gradient(t), self.half)
        g_dev = to_device(g, self.half)
        g_keep = g_dev.clone()
        if t % self.wl.T == 0:
            self.refresh(g, g_dev)
        self.gst.step(self.w_dev, g_dev)
        self.w_ref = orc.oracle_step(self.ost, self.w_ref, g, refresh=False)
        torch.cuda.synchronize()
        assert torch.equal(g_keep, g_dev), "the step must not modify the gradient"
        if check:
            self.compare()

    def compare(self):
        gst, ost = self.gst, self.ost
        pairs = [
            ("core", gst.export(B.WHAT_CORE), ost.core),
            ("n_l", gst.export(B.WHAT_N_L), ost.n_l),
            ("m_l", gst.export(B.WHAT_M_L), ost.m_l),
            ("v_l", gst.export(B.WHAT_V_L), ost.v_l),
        ]
        if self.wl.k > 0:
            pairs += [
                ("n_s", gst.export(B.WHAT_N_S), ost.n_s),
                ("m_s", gst.export(B.WHAT_M_S), ost.m_s),
                ("v_s", gst.export(B.WHAT_V_S), ost.v_s),
            ]
        for name, a, b in pairs:
            e = H.rel_err(a, b)
            self._note(name, e)
            assert e <= TOL_FLOAT, f"{name}: max relative error {e} at t={ost.t - 1}"
        w_gpu = from_device(self.w_dev, self.half)
        if self.half:
            # fp16 storage: 1e-4 is below half-precision resolution; compare in ulps
            a = synth.to_half_pairs(w_gpu).view(np.int16).astype(np.int32)
            b = synth.to_half_pairs(self.w_ref).view(np.int16).astype(np.int32)
            d = np.abs(a - b)
            assert d.max() <= 1, f"weights differ by {d.max()} fp16 ulps"
            frac = float(np.mean(d == 0))
            self._note("w_mismatch_frac", 1.0 - frac)
            assert frac >= 0.999, f"only {frac} of the fp16 weights are bit-identical"
            self.w_ref = w_gpu          # follow the GPU's rounding so one-ulp choices do not compound
        else:
            e = H.rel_err(w_gpu, self.w_ref)
            self._note("w", e)
            assert e <= TOL_FLOAT, f"weights: max relative error {e}"
