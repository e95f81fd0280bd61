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

TOL_FLOAT = 1e-4       # max relative error, entries measured against max(|ref|, 2^-7 rms(ref)); see helpers.rel_err
TOL_FRO = 5e-6         # and the whole array: ||a - b||_F / ||b||_F (split-TF32 products carry 2^-21 relative error
                       # each, and an entry passes through up to 2 N of them)
TOL_GRAM = 2e-4        # largest entry error of a Gram matrix over its largest diagonal entry
TOL_ANGLE = 1e-3       # largest principal-angle sine of a refreshed factor
TOL_ORTHO = 1e-5       # max |U^H U - I|


def to_device(x: np.ndarray, half) -> torch.Tensor:
    """complex64 array -> device tensor in the storage layout (float32, float16 or bfloat16 pairs; `half` is False,
    True or "bf16")."""
    if half == "bf16":
        return torch.from_numpy(synth.to_bf16_pairs(x).view(np.int16)).cuda()
    if half:
        return torch.from_numpy(synth.to_half_pairs(x)).cuda()
    return torch.from_numpy(np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,))).cuda()


def from_device(t: torch.Tensor, half) -> np.ndarray:
    a = t.cpu().numpy()
    if half == "bf16":
        return synth.from_bf16_pairs(a.view(np.uint16))
    if half:
        return synth.from_half_pairs(a)
    return np.ascontiguousarray(a).view(np.complex64)[..., 0]


def half_ordinals(x: np.ndarray, half=True) -> np.ndarray:
    """fp16 (or bfloat16) (re, im) pairs of a complex array as integers that count representable values along the real
    line (sign-magnitude bit patterns mapped to a monotone scale; +0 and -0 coincide): differences are distances in ulps."""
    bits = (synth.to_bf16_pairs(x) if half == "bf16" else synth.to_half_pairs(x).view(np.uint16)).astype(np.int32)
    mag = bits & 0x7FFF
    return np.where(bits & 0x8000, -mag, mag)


def storage_exact(x: np.ndarray, half) -> np.ndarray:
    if half == "bf16":
        return synth.from_bf16_pairs(synth.to_bf16_pairs(x))
    return synth.from_half_pairs(synth.to_half_pairs(x)) if half else x


class Pair:
    def __init__(self, wl: synth.Workload, tensor_id=0, warm_refresh=False, stagewise_w=False, hooi_iters=0, **over):
        # stagewise_w: the expected weight is the oracle's weight update applied to the GPU's own normalised
        # updates N_L, N_S (which are themselves checked against the oracle's formula on the GPU's moments, and the
        # moments against the oracle's).  Needed where core entries vanish by construction: for a matrix the
        # refreshed factors are its singular vectors, so on the refresh step the off-diagonal core entries are
        # pure rounding noise, and N = M / (sqrt(V) + eps) turns that noise into unit-size numbers on both sides.
        self.stagewise_w = stagewise_w
        self.wl = wl
        self.src = synth.GradientSource(wl, tensor_id)
        kw = dict(lr=wl.lr, alpha=1.0, lam=1.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
        kw.update(over)
        self.half = "bf16" if wl.bf16_storage else wl.half_storage
        self.ocfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, half_storage=wl.half_storage,
                                     bf16_storage=wl.bf16_storage, hooi_iters=hooi_iters, hooi_warm=warm_refresh, **kw)
        self.ost = orc.OracleState(self.ocfg)
        self.gcfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, half_storage=wl.half_storage,
                                  bf16_storage=wl.bf16_storage, auto_refresh=False,
                                  warm_refresh=warm_refresh, hooi_iters=hooi_iters, **kw)
        self.gst = B.TgradState(self.gcfg)
        w0 = storage_exact(self.src.weight(), self.half)
        self.w_ref = w0
        self.w_dev = to_device(w0, self.half)
        self.report = {}

    def _note(self, name, val):
        self.report[name] = max(self.report.get(name, 0.0), float(val))

    def _note_min(self, name, val):
        self.report[name] = min(self.report.get(name, 1e9), float(val))

    def sync_oracle_from_gpu(self):
        """Snapshot parity: the oracle takes over the whole exported GPU state (counter, Omega, factors, all
        four moments, weight), so that its next step starts from exactly what the GPU's next step starts from."""
        gst, ost = self.gst, self.ost
        flags, t, _ = gst.query_status()
        assert flags == 0, f"sticky flags {flags}"
        ost.t = t
        ost.factors = gst.factors()
        ost.m_l, ost.v_l = gst.export(B.WHAT_M_L), gst.export(B.WHAT_V_L)
        if self.wl.k > 0:
            ost.omega = gst.export(B.WHAT_OMEGA)
            ost.m_s, ost.v_s = gst.export(B.WHAT_M_S), gst.export(B.WHAT_V_S)
        else:
            ost.omega = np.zeros(0, np.uint32)
        self.w_ref = from_device(self.w_dev, self.half)

    def refresh(self, g: np.ndarray, g_dev: torch.Tensor):
        before = g_dev.clone()
        self.gst.refresh_subspace(g_dev)
        flags, _, sweeps = self.gst.query_status()
        assert flags == 0, f"sticky flags {flags}, sweeps {sweeps}"
        assert torch.equal(before, g_dev), "refresh must leave the gradient as it found it"
        orc.oracle_refresh(self.ost, g)
        om = self.gst.export(B.WHAT_OMEGA)
        lr_first = self.ocfg.composition == "lr_us"
        if not lr_first:
            assert np.array_equal(om, self.ost.omega), "Omega differs from the oracle"
        if self.ocfg.composition == "us_lr" and self.ocfg.hooi_iters == 0 and self.ocfg.strategy == "topk":
            # the Gram matrices themselves, entry by entry, against the definition R_(n) R_(n)^H in complex128
            # (fp32 storage: TF32 inputs on the long contractions, hence 2e-4 of the largest diagonal entry)
            res = orc.residual(g, self.ost.omega).astype(np.complex128)
            for n in range(len(self.wl.shape)):
                want = orc.mode_gram(res, n)
                got = self.gst.export(B.WHAT_GRAM_BASE + n).astype(np.complex128)
                scale = float(np.abs(np.diag(want)).max())
                if scale > 0:
                    e = float(np.abs(got - want).max() / scale)
                    self._note("gram", e)
                    assert e <= TOL_GRAM, f"mode {n}: Gram matrix off by {e} of its largest diagonal entry"
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
        if lr_first and self.wl.k > 0:
            # Low rank first: Omega is chosen from G - P_U(G), which the two sides compute in different arithmetic, so
            # entries whose key sits at the threshold may legitimately fall on either side.  Compared: the sets agree
            # except for such entries (keys of the oracle's residual under the GPU's factors within 1e-3 of the
            # threshold, and few of them); then the oracle takes the GPU's set, as it takes its factors.
            c = self.ocfg
            res = orc.lowrank_residual(c, g, self.ost.factors)
            key = orc.selection_key(res, c.strategy, c.seed, (self.ost.t // c.T)).astype(np.float64)
            want = orc.sparse_indices(res, c.k, c.strategy, c.seed, self.ost.t // c.T)
            thr = np.sort(key)[-c.k]
            diff = np.setxor1d(om.astype(np.int64), want.astype(np.int64))
            self._note("omega_boundary_entries", diff.size)
            assert om.size == c.k and np.all(np.diff(om.astype(np.int64)) > 0)
            assert diff.size <= max(2, c.k // 100), f"{diff.size} of {c.k} indices differ"
            if diff.size:
                assert np.max(np.abs(key[diff] - thr)) <= 1e-3 * thr, "an index away from the threshold differs"
            self.ost.omega = om.copy()
        return sweeps

    def step(self, t: int, check=True):
        g = storage_exact(self.src.gradient(t), self.half)
        g_dev = to_device(g, self.half)
        g_keep = g_dev.clone()
        if t % self.wl.T == 0:
            self.refresh(g, g_dev)
        self.gst.step(self.w_dev, g_dev)
        self.w_prev = self.w_ref
        self.w_ref = orc.oracle_step(self.ost, self.w_ref, g, refresh=False)
        torch.cuda.synchronize()
        assert torch.equal(g_keep, g_dev), "the step must not modify the gradient"
        if check:
            self.compare()

    def compare(self):
        gst, ost = self.gst, self.ost
        t = ost.t - 1
        c = self.ocfg
        m_l, v_l = gst.export(B.WHAT_M_L), gst.export(B.WHAT_V_L)
        pairs = [
            ("core", gst.export(B.WHAT_CORE), ost.core),
            ("m_l", m_l, ost.m_l),
            ("v_l", v_l, ost.v_l),
        ]
        # N = M^/(sqrt(V^)+eps) has unit scale whatever the size of the entry, so a core entry that
        # is tiny by cancellation has an ill-conditioned N: check N against the oracle's formula
        # evaluated on the GPU's own moments (tight), and the moments against the oracle's.
        dirs = [("n_l", gst.export(B.WHAT_N_L), orc.adam_direction(m_l, v_l, c.beta1, c.beta2, c.eps, t))]
        if self.wl.k > 0:
            m_s, v_s = gst.export(B.WHAT_M_S), gst.export(B.WHAT_V_S)
            pairs += [("m_s", m_s, ost.m_s), ("v_s", v_s, ost.v_s)]
            dirs.append(("n_s", gst.export(B.WHAT_N_S), orc.adam_direction(m_s, v_s, c.beta1, c.beta2, c.eps, t)))
        for name, a, b in dirs:
            e = float(np.max(np.abs(a - b) / np.maximum(np.abs(b), 1e-30))) if a.size else 0.0
            self._note(name, e)
            assert e <= 1e-5, f"{name}: max relative error {e} at t={t}"
        for name, a, b in pairs:
            e = H.rel_err(a, b)
            self._note(name, e)
            assert e <= TOL_FLOAT, f"{name}: max relative error {e} at t={ost.t - 1}"
            # the same metric at the floor 1e-3 rms: asserted where the quantity is element-wise (the sparse
            # moments), reported for the contracted quantities together with the tightest passing floor
            e3 = H.rel_err(a, b, H.FLOOR_CONTRACT)
            self._note(name + "@1e-3", e3)
            if name in ("m_s", "v_s") and c.composition != "lr_us":       # (low rank first: the sparse values are differences too)
                assert e3 <= TOL_FLOAT, f"{name}: max relative error {e3} at the 1e-3 rms floor"
            elif a.size <= (1 << 22):
                self._note_min(name + "_floor_log2", H.tightest_floor_log2(a, b, TOL_FLOAT, lo=7))
                self._note(name + "_below_1e-3", H.below_floor_fraction(b))
            f = H.fro_err(a, b)
            self._note(name + "_fro", f)
            assert f <= TOL_FRO, f"{name}: Frobenius error {f} at t={ost.t - 1}"
        w_gpu = from_device(self.w_dev, self.half)
        if self.stagewise_w:
            n_s_gpu = gst.export(B.WHAT_N_S) if self.wl.k > 0 else np.zeros(0, np.complex64)
            self.w_ref = orc.weight_update(c, self.w_prev, gst.export(B.WHAT_N_L), n_s_gpu, ost.omega, ost.factors)
        if self.half:
            # fp16 storage: 1e-4 is below half-precision resolution; compare in ulps
            d = np.abs(half_ordinals(w_gpu, self.half) - half_ordinals(self.w_ref, self.half))
            # an update that cancels the old weight leaves a number far below the ulp of its operands, where both
            # sides hold fp32 rounding noise: such an entry is within one ulp *of the old weight*
            def parts(x):
                return np.ascontiguousarray(x).view(np.float32).reshape(x.shape + (2,))
            old = np.abs(parts(self.w_prev))
            ulp_old = (np.spacing(old) * 65536.0) if self.half == "bf16" else np.spacing(old.astype(np.float16)).astype(np.float32)
            cancelled = np.abs(parts(w_gpu) - parts(self.w_ref)) <= ulp_old
            d = np.where(cancelled & (d > 1), 1, d)
            assert d.max() <= 1, f"weights differ by {d.max()} ulps of the 16-bit storage type"
            frac = float(np.mean(d == 0))
            self._note("w_mismatch_frac", 1.0 - frac)
            assert frac >= 0.999, f"only {frac} of the fp16 weights are bit-identical"
            self.w_ref = w_gpu          # follow the GPU's rounding so one-ulp choices do not compound
        else:
            e = H.rel_err(w_gpu, self.w_ref, H.FLOOR_CONTRACT)
            self._note("w@1e-3", e)
            assert e <= TOL_FLOAT, f"weights: max relative error {e} at the 1e-3 rms floor"
        assert gst.query_status()[0] == 0, "sticky device flags after a step"


# ---------------------------------------------------------------------------------------------
# Full-size checks on sampled outputs: each sampled value is computed by the oracle's own
# functions on a slice of the problem, using linearity of the mode products.
# ---------------------------------------------------------------------------------------------

def omega_properties(g: np.ndarray, omega: np.ndarray, k: int):
    """The definition of the top-k set restated as properties that can be checked in linear
    time at any size: size k, strictly ascending, every key inside >= every key outside, and
    among keys equal to the threshold the chosen ones are the lowest flat indices."""
    key = orc.magnitude_key(g).reshape(-1)
    om = omega.astype(np.int64)
    assert om.size == k
    if k == 0:
        return
    assert np.all(np.diff(om) > 0) and om[0] >= 0 and om[-1] < key.size
    inside = np.zeros(key.size, dtype=bool)
    inside[om] = True
    thr = key[om].min()
    assert key[~inside].max(initial=-1.0) <= thr
    eq = np.flatnonzero(key == thr)
    eq_in = inside[eq]
    n_in = int(eq_in.sum())
    assert np.all(eq_in[:n_in]) and not np.any(eq_in[n_in:]), "ties must go to the lower flat index"
    assert int((key > thr).sum()) + n_in == k


def core_entry(r: np.ndarray, factors, j):
    """One entry of R x_1 U1^H ... x_N UN^H, summed over slices of the first mode."""
    cols = [np.ascontiguousarray(u[:, jj:jj + 1]) for u, jj in zip(factors, j)]
    acc = 0.0 + 0.0j
    for i1 in range(r.shape[0]):
        part = orc.tucker_compress(r[i1], cols[1:]).reshape(())
        acc += np.conj(complex(cols[0][i1, 0])) * complex(part)
    return acc


def dense_update_entry(n_l: np.ndarray, factors, idx):
    """One entry of N_L x_1 U1 ... x_N UN."""
    rows = [np.ascontiguousarray(u[i:i + 1, :]) for u, i in zip(factors, idx)]
    return complex(orc.tucker_reconstruct(n_l, rows).reshape(()))


def gram_entry(r: np.ndarray, n: int, a: int, b: int):
    sub = np.take(r, [a, b], axis=n)
    return complex(orc.mode_gram(sub, n)[0, 1])


def full_core_by_slices(r: np.ndarray, factors) -> np.ndarray:
    """R x_1 U1^H ... x_N UN^H in complex128 without a complex128 copy of R: the leading mode is summed slice by
    slice (linearity), and inside a slice the modes are contracted last-first with the oracle's mode product
    (mode products commute; the oracle's pins check that on small tensors)."""
    uh = [np.conj(np.asarray(u, dtype=np.complex128)).T for u in factors]
    core = np.zeros([u.shape[1] for u in factors], dtype=np.complex128)
    nd = r.ndim - 1
    for i1 in range(r.shape[0]):
        x = np.asarray(r[i1], dtype=np.complex128)
        for n in range(nd - 1, -1, -1):
            x = orc.mode_n_product(x, uh[n + 1], n)
        core += uh[0][:, i1].reshape((-1,) + (1,) * nd) * x[None]
    return core


def dense_update_slab(n_l: np.ndarray, factors, lead):
    """The trailing A x B slab at leading indices `lead` of N_L x_1 U1 ... x_N UN: one reconstruction call of the
    oracle on factors whose leading modes are cut down to the wanted row."""
    fs = [np.ascontiguousarray(u[i:i + 1, :]) for u, i in zip(factors, lead)] + list(factors[len(lead):])
    return orc.tucker_reconstruct(n_l, fs).reshape(factors[-2].shape[0], factors[-1].shape[0])


class SampledChecker:
    """Refresh + steps at a size where a full oracle step is out of reach (the 545 M-entry configuration): Omega
    by its defining properties, sampled Gram entries, the factors against an eigen-decomposition of the exported
    Gram matrices, the whole compressed gradient, both Adam updates in full, and the updated weight on whole
    slabs (first slabs, every slab of the last leading index -- which holds the partly filled last round of the
    streaming kernels -- and random ones), every entry compared."""

    def __init__(self, wl: synth.Workload, tensor_id=0, n_samples=6, n_random_slabs=64, seed=0, warm_refresh=False):
        self.wl = wl
        self.half = wl.half_storage
        self.src = synth.GradientSource(wl, tensor_id)
        self.cfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, lr=wl.lr, half_storage=self.half, auto_refresh=False,
                                 warm_refresh=warm_refresh)
        self.st = B.TgradState(self.cfg)
        self.w = storage_exact(self.src.weight(), self.half)
        self.w_dev = to_device(self.w, self.half)
        self.rng = np.random.default_rng(seed)
        self.n_samples = n_samples
        self.n_random_slabs = n_random_slabs
        self.t = 0
        self.m_l = np.zeros(wl.ranks, np.complex64); self.v_l = np.zeros(wl.ranks, np.float32)
        self.m_s = np.zeros(wl.k, np.complex64); self.v_s = np.zeros(wl.k, np.float32)
        self.report = {}

    def _note(self, name, val):
        self.report[name] = max(self.report.get(name, 0.0), float(val))

    def refresh(self, g, g_dev):
        wl = self.wl
        self.st.refresh_subspace(g_dev)
        flags, _, sweeps = self.st.query_status()
        assert flags == 0, (flags, sweeps)
        self.report["sweeps"] = sweeps
        self.omega = self.st.export(B.WHAT_OMEGA)
        omega_properties(g, self.omega, wl.k)
        r = orc.residual(g, self.omega)
        self.factors = self.st.factors()
        for n in range(len(wl.shape)):
            a_gpu = self.st.export(B.WHAT_GRAM_BASE + n).astype(np.complex128)
            scale = float(np.max(np.abs(np.diag(a_gpu))))
            for _ in range(self.n_samples):
                a, b = (int(x) for x in self.rng.integers(0, wl.shape[n], 2))
                want = gram_entry(r, n, a, b) if a != b else complex(orc.mode_gram(np.take(r, [a], axis=n), n)[0, 0])
                self._note("gram", abs(a_gpu[a, b] - want) / scale)
                assert abs(a_gpu[a, b] - want) <= 1e-5 * scale, (n, a, b)
            assert np.allclose(a_gpu, np.conj(a_gpu).T)
            w, v = np.linalg.eigh(a_gpu)
            top = v[:, ::-1][:, :wl.ranks[n]]
            ang = H.max_sin_angle(self.factors[n], top)
            self._note("angle", ang)
            assert ang <= TOL_ANGLE, (n, ang)
            od = H.ortho_defect(self.factors[n])
            self._note("ortho", od)
            assert od <= TOL_ORTHO, (n, od)
        return r

    def _slab_list(self):
        wl = self.wl
        lead_shape = wl.shape[:-2]
        nslab = int(np.prod(lead_shape))
        per_last = nslab // lead_shape[0]
        picks = set(range(min(4, nslab)))
        picks.update(range(nslab - per_last, nslab))                    # every slab of the last leading index
        picks.update(int(x) for x in self.rng.integers(0, nslab, self.n_random_slabs))
        return sorted(picks), lead_shape

    def step(self, refresh=False):
        wl, t = self.wl, self.t
        g = storage_exact(self.src.gradient(t), self.half)
        g_dev = to_device(g, self.half)
        if t % wl.T == 0 or refresh:
            r = self.refresh(g, g_dev)
        else:
            r = orc.residual(g, self.omega)
        self.st.step(self.w_dev, g_dev)
        torch.cuda.synchronize()
        st = self.st
        assert st.query_status()[0] == 0
        # compressed gradient: every entry
        core = st.export(B.WHAT_CORE)
        want_core = full_core_by_slices(r, self.factors)
        e = H.rel_err(core, want_core, H.FLOOR_FRAC_LARGE); self._note("core", e); assert e <= TOL_FLOAT, ("core", e)
        f = H.fro_err(core, want_core); self._note("core_fro", f); assert f <= TOL_FRO, ("core", f)
        self._note("core@1e-3", H.rel_err(core, want_core, H.FLOOR_CONTRACT))
        del r
        # both Adam updates in full (element-wise), from the GPU's own compressed inputs
        n_l, self.m_l, self.v_l = orc.adam_update(core, self.m_l, self.v_l, 0.9, 0.999, 1e-8, t)
        for name, a, b in (("n_l", st.export(B.WHAT_N_L), n_l), ("m_l", st.export(B.WHAT_M_L), self.m_l),
                           ("v_l", st.export(B.WHAT_V_L), self.v_l)):
            e = H.rel_err(a, b); self._note(name, e); assert e <= TOL_FLOAT, (name, e)
        g_s = orc.sparse_gather(g, self.omega)
        n_s, self.m_s, self.v_s = orc.adam_update(g_s, self.m_s, self.v_s, 0.9, 0.999, 1e-8, t)
        n_s_gpu = st.export(B.WHAT_N_S)
        for name, a, b in (("n_s", n_s_gpu, n_s), ("m_s", st.export(B.WHAT_M_S), self.m_s),
                           ("v_s", st.export(B.WHAT_V_S), self.v_s)):
            e = H.rel_err(a, b, H.FLOOR_CONTRACT); self._note(name, e); assert e <= TOL_FLOAT, (name, e)
        # weights: whole slabs, every entry
        w_new = from_device(self.w_dev, self.half)
        n_l_gpu = st.export(B.WHAT_N_L)
        lr = float(np.float32(wl.lr))
        om = self.omega.astype(np.int64)
        slabs, lead_shape = self._slab_list()
        E = wl.shape[-2] * wl.shape[-1]
        n_checked = n_same = 0
        w_rms = float(np.sqrt(np.mean(np.abs(self.w[tuple(0 for _ in lead_shape)].astype(np.complex128)) ** 2)))
        for s_ in slabs:
            lead = np.unravel_index(s_, lead_shape)
            d = dense_update_slab(n_l_gpu, self.factors, lead)
            want = self.w[lead].astype(np.complex128) - lr * d
            j0, j1 = np.searchsorted(om, [s_ * E, (s_ + 1) * E])
            loc = om[j0:j1] - s_ * E
            if self.half:
                want = synth.from_half_pairs(synth.to_half_pairs(want.astype(np.complex64))).astype(np.complex128)
                wf = want.reshape(-1)
                wf[loc] = wf[loc] - lr * n_s_gpu[j0:j1].astype(np.complex128)
                dd = np.abs(half_ordinals(w_new[lead]) - half_ordinals(want.astype(np.complex64)))
                # same rule as the element-wise comparison: where the update cancels the old weight, one ulp *of the
                # old weight* is the resolution of both sides
                def parts(x):
                    return np.ascontiguousarray(x.astype(np.complex64)).view(np.float32).reshape(x.shape + (2,))
                ulp_old = np.spacing(np.abs(parts(self.w[lead])).astype(np.float16)).astype(np.float32)
                cancelled = np.abs(parts(w_new[lead]) - parts(want)) <= ulp_old
                dd = np.where(cancelled & (dd > 1), 1, dd)
                if dd.max() > 1:
                    bad = np.argwhere(dd > 1)[0]
                    flat = int(bad[0]) * wl.shape[-1] + int(bad[1])
                    raise AssertionError((lead, int(dd.max()), tuple(int(x) for x in bad), "in Omega" if flat in set(loc.tolist()) else "dense",
                                          complex(self.w[lead][bad[0], bad[1]]), complex(w_new[lead][bad[0], bad[1]]),
                                          complex(want[bad[0], bad[1]])))
                n_checked += dd.size; n_same += int((dd == 0).sum())
            else:
                wf = want.reshape(-1)
                wf[loc] = wf[loc] - lr * n_s_gpu[j0:j1].astype(np.complex128)
                err = np.max(np.abs(w_new[lead] - want) / np.maximum(np.abs(want), H.FLOOR_CONTRACT * w_rms))
                self._note("w", err)
                assert err <= TOL_FLOAT, (lead, err)
        if self.half:
            self._note("w_mismatch_frac", 1.0 - n_same / n_checked)
            assert n_same >= 0.999 * n_checked
        self.report["slabs_checked"] = len(slabs)
        self.w = w_new
        self.t += 1
