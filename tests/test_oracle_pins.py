"""Pins for the CPU oracle: brute force, closed forms, invariants and the
worked example the paper prints.  None of these re-type an oracle formula."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import tgrad_oracle as orc
from paper_2501_02379_b200 import synth
from tests import helpers as H

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---- top-k: brute force, ties, edge k -----------------------------------------------------

@pytest.mark.parametrize("seed", [0, 1, 2])
@pytest.mark.parametrize("k", [0, 1, 7, 59, 60])
def test_topk_brute_force_with_ties(seed, k):
    g = synth.quantised_ties((3, 4, 5), 2, seed)          # 60 entries on a 5x5 grid: many ties
    got = orc.sparse_indices_topk(g, k)
    assert got.dtype == np.uint32
    assert got.tolist() == H.brute_topk(g, k)


def test_topk_brute_force_random():
    rng = np.random.default_rng(5)
    g = (rng.standard_normal((4, 8, 8, 4)) + 1j * rng.standard_normal((4, 8, 8, 4))).astype(np.complex64)
    for k in (1, 100, 1023, 1024):
        assert orc.sparse_indices_topk(g, k).tolist() == H.brute_topk(g, k)


def test_topk_all_equal_takes_lowest_indices():
    g = np.full((5, 6), 1 + 1j, dtype=np.complex64)
    assert orc.sparse_indices_topk(g, 11).tolist() == list(range(11))


def test_key_is_unfused_fp32():
    # re*re + im*im where an FMA would round differently: choose values whose
    # product needs more than 24 bits.
    re = np.float32(1.0 + 2.0 ** -12)
    im = np.float32(2.0 ** -13 + 2.0 ** -25)
    g = np.array([complex(re, im)], dtype=np.complex64)
    want = np.float32(np.float32(re * re) + np.float32(im * im))
    exact = float(re) ** 2 + float(im) ** 2
    assert orc.magnitude_key(g)[0] == want
    assert orc.magnitude_key(g).dtype == np.float32
    # sanity: the unfused result is what separately rounded ops give, and is a float32
    assert abs(float(want) - exact) <= 2.0 ** -22


def test_planted_outliers_are_selected():
    wl = synth.WORKLOADS["cfg1"]
    src = synth.GradientSource(wl)
    g = src.gradient(0)
    om = orc.sparse_indices_topk(g, wl.k)
    assert wl.k == 1475
    assert np.array_equal(om.astype(np.int64), np.sort(src.out_pos))
    r = orc.residual(g, om)
    gs = orc.sparse_gather(g, om)
    back = r.copy().reshape(-1)
    assert np.all(back[om.astype(np.int64)] == 0)
    back[om.astype(np.int64)] += gs
    assert np.array_equal(back.view(np.float32), g.reshape(-1).view(np.float32))     # bitwise


# ---- mode products / projection ---------------------------------------------------------------

def test_mode_product_matches_definition_loops():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((3, 4, 2)) + 1j * rng.standard_normal((3, 4, 2))
    for n in range(3):
        u = rng.standard_normal((5, x.shape[n])) + 1j * rng.standard_normal((5, x.shape[n]))
        got = orc.mode_n_product(x, u, n)
        shp = list(x.shape); shp[n] = 5
        want = np.zeros(shp, dtype=np.complex128)
        for idx in itertools.product(*[range(s) for s in shp]):
            acc = 0
            for i in range(x.shape[n]):
                src = list(idx); src[n] = i
                acc += x[tuple(src)] * u[idx[n], i]
            want[idx] = acc
        assert np.allclose(got, want, atol=1e-12)


def test_unfold_column_order_first_index_fastest():
    x = np.arange(24).reshape(2, 3, 4).astype(np.complex128)
    m = orc.unfold(x, 1)
    # column j = i_1 + I_1 * i_3 (0-based) for mode 2 of a 3-way tensor
    for i1 in range(2):
        for i3 in range(4):
            assert np.array_equal(m[:, i1 + 2 * i3], x[i1, :, i3])
    # property (U x_k A)_(k) = U A_(k)
    rng = np.random.default_rng(1)
    u = rng.standard_normal((5, 3))
    assert np.allclose(orc.unfold(orc.mode_n_product(x, u, 1), 1), u @ m)


def test_projection_idempotent_and_order_free():
    rng = np.random.default_rng(2)
    shape, ranks = (6, 5, 4, 3), (3, 2, 2, 2)
    us = [H.random_orthonormal(rng, i, r) for i, r in zip(shape, ranks)]
    for u in us:
        assert H.ortho_defect(u) < 1e-13
    c = rng.standard_normal(ranks) + 1j * rng.standard_normal(ranks)
    assert np.allclose(orc.tucker_compress(orc.tucker_reconstruct(c, us), us), c, atol=1e-12)
    x = rng.standard_normal(shape) + 1j * rng.standard_normal(shape)
    p1 = orc.tucker_reconstruct(orc.tucker_compress(x, us), us)
    p2 = orc.tucker_reconstruct(orc.tucker_compress(p1, us), us)
    assert np.allclose(p1, p2, atol=1e-12)
    # any order of the mode products gives the same core
    base = orc.tucker_compress(x, us)
    for perm in itertools.permutations(range(4)):
        y = x
        for n in perm:
            y = orc.mode_n_product(y, np.conj(us[n]).T, n)
        assert np.allclose(y, base, atol=1e-12)
    # explicit 4-fold sum for one core entry (conjugated factors)
    j = (1, 1, 0, 1)
    acc = 0
    for idx in itertools.product(*[range(s) for s in shape]):
        f = 1
        for n in range(4):
            f *= np.conj(us[n][idx[n], j[n]])
        acc += x[idx] * f
    assert abs(acc - base[j]) < 1e-12


def test_exact_tucker_recovery_no_sparse():
    rng = np.random.default_rng(3)
    shape, ranks = (7, 6, 5, 4), (3, 2, 2, 2)
    a = [H.random_orthonormal(rng, i, r) for i, r in zip(shape, ranks)]
    c = rng.standard_normal(ranks) + 1j * rng.standard_normal(ranks)
    x = orc.tucker_reconstruct(c, a)
    us = orc.tucker_factors(x, ranks)
    for u, an in zip(us, a):
        assert H.max_sin_angle(u, an) < 1e-6
        assert H.ortho_defect(u) < 1e-6
    us64 = [u.astype(np.complex128) for u in us]
    back = orc.tucker_reconstruct(orc.tucker_compress(x, us64), us64)
    assert H.fro_err(back, x) < 1e-6


def test_exact_recovery_with_outliers_on_zero_slices():
    rng = np.random.default_rng(4)
    shape, ranks = (8, 6, 5, 4), (3, 2, 2, 2)
    a = [H.random_orthonormal(rng, i, r) for i, r in zip(shape, ranks)]
    a[0][6:, :] = 0                                # rows 6,7 of mode 1: low-rank part vanishes there
    q, _ = np.linalg.qr(a[0][:6]); a[0][:6] = q
    c = rng.standard_normal(ranks) + 1j * rng.standard_normal(ranks)
    low = orc.tucker_reconstruct(c, a)
    g = low.copy()
    k = 9
    pos = rng.choice(2 * 6 * 5 * 4, size=k, replace=False) + 6 * (6 * 5 * 4)
    g.reshape(-1)[pos] = 100.0 * np.exp(1j * rng.uniform(0, 6.28, k))
    g = g.astype(np.complex64)
    om = orc.sparse_indices_topk(g, k)
    assert np.array_equal(om.astype(np.int64), np.sort(pos))
    r = orc.residual(g, om)
    assert H.fro_err(r, low) < 1e-6
    us = [u.astype(np.complex128) for u in orc.tucker_factors(r, ranks)]
    rec = np.ascontiguousarray(orc.tucker_reconstruct(orc.tucker_compress(r, us), us))
    rec.reshape(-1)[om.astype(np.int64)] += orc.sparse_gather(g, om)
    assert H.fro_err(rec, g) < 1e-5


def test_matrix_case_is_svd():
    rng = np.random.default_rng(6)
    m = rng.standard_normal((9, 7)) + 1j * rng.standard_normal((9, 7))
    u1, u2 = orc.tucker_factors(m, (3, 2))
    uu, s, vh = np.linalg.svd(m)
    assert H.max_sin_angle(u1, uu[:, :3]) < 1e-6
    # mode-2 unfolding is M^T = conj(V) S U^T: its left singular vectors are conj(V) = (V^H)^T
    assert H.max_sin_angle(u2, vh[:2].T) < 1e-6
    # full-rank factors: the core carries the singular values (|core| is diag(s) up to phases)
    f1, f2 = orc.tucker_factors(m, (7, 7))
    core = orc.tucker_compress(m, [f1.astype(np.complex128), f2.astype(np.complex128)])
    assert np.allclose(np.sort(np.abs(np.diag(core)))[::-1], s, rtol=1e-5)
    off = core - np.diag(np.diag(core))
    assert np.max(np.abs(off)) < 1e-5 * s[0]


def test_gram_identities_and_eigen_residual():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((5, 4, 3, 6)) + 1j * rng.standard_normal((5, 4, 3, 6))
    fro2 = float(np.sum(np.abs(x) ** 2))
    for n in range(4):
        a = orc.mode_gram(x, n)
        assert np.allclose(a, np.conj(a).T)
        assert abs(np.trace(a).real - fro2) < 1e-10 * fro2      # ||X||_F = ||X_(n)||_F
        # one entry by explicit loops
        acc = 0
        for idx in itertools.product(*[range(s) for s in x.shape]):
            if idx[n] == 1:
                other = list(idx); other[n] = 2
                acc += x[idx] * np.conj(x[tuple(other)])
        assert abs(acc - a[1, 2]) < 1e-10
        us = orc.tucker_factors(x, [x.shape[m] for m in range(4)])
        u = us[n].astype(np.complex128)
        lam = np.real(np.einsum("ij,ik,kj->j", np.conj(u), a, u))
        assert np.all(np.diff(lam) <= 1e-4 * lam[0])            # descending
        assert np.linalg.norm(a @ u - u * lam) < 1e-5 * np.linalg.norm(a)
        assert abs(lam.sum() - fro2) < 1e-5 * fro2
        # canonical phase: largest-modulus component of every column is real positive
        for j in range(u.shape[1]):
            i = np.argmax(np.abs(u[:, j]))
            assert abs(u[i, j].imag) < 1e-6 and u[i, j].real > 0


# ---- refinement of the factors (higher-order orthogonal iteration) --------------------------------

def _recon_error(x, us):
    return float(np.linalg.norm(x - orc.tucker_reconstruct(orc.tucker_compress(x, us), us)))


def test_hooi_never_increases_the_reconstruction_error():
    # each mode update maximises the energy kept given the other factors, so || R - P_U R ||_F cannot grow from sweep
    # to sweep, and it starts from the truncated-SVD factors' error
    rng = np.random.default_rng(31)
    shape, ranks = (7, 6, 5, 4), (3, 2, 2, 2)
    x = (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)      # no low-rank structure
    errs = [_recon_error(x, orc.tucker_factors_hooi(x, ranks, it)) for it in range(5)]
    assert errs[0] == pytest.approx(_recon_error(x, orc.tucker_factors(x, ranks)), rel=1e-12)
    for a, b in zip(errs, errs[1:]):
        assert b <= a * (1 + 1e-6)
    assert errs[-1] < errs[0] * 0.999          # and on an unstructured tensor the refinement does help
    for u in orc.tucker_factors_hooi(x, ranks, 3):
        assert H.ortho_defect(u) < 1e-6
        for j in range(u.shape[1]):
            i = np.argmax(np.abs(u[:, j]))
            assert abs(u[i, j].imag) < 1e-6 and u[i, j].real > 0


def test_hooi_fixed_point_on_an_exactly_low_rank_tensor():
    rng = np.random.default_rng(32)
    shape, ranks = (8, 7, 6), (3, 2, 2)
    us = [H.random_orthonormal(rng, i, r) for i, r in zip(shape, ranks)]
    c = rng.standard_normal(ranks) + 1j * rng.standard_normal(ranks)
    x = orc.tucker_reconstruct(c, us)
    f0 = orc.tucker_factors(x, ranks)
    f2 = orc.tucker_factors_hooi(x, ranks, 2)
    for a, b, planted in zip(f0, f2, us):
        assert H.max_sin_angle(b, planted) < 1e-6 and H.max_sin_angle(a, b) < 1e-6
    assert _recon_error(x, f2) < 1e-6 * np.linalg.norm(x)


def test_hooi_on_a_matrix_stays_at_the_svd():
    rng = np.random.default_rng(33)
    x = rng.standard_normal((9, 7)) + 1j * rng.standard_normal((9, 7))
    u, s_, vh = np.linalg.svd(x)
    f = orc.tucker_factors_hooi(x, (3, 3), 3)
    assert H.max_sin_angle(f[0], u[:, :3]) < 1e-6
    assert H.max_sin_angle(f[1], np.conj(vh[:3]).T.conj()) < 1e-6


def test_hooi_update_is_the_best_subspace_for_the_other_factors():
    # the defining property of one mode update: with the other factors fixed, no other orthonormal I_n x r_n matrix
    # keeps more energy || R x_1 U1^H .. x_N UN^H ||_F
    rng = np.random.default_rng(34)
    shape, ranks = (6, 5, 4), (2, 2, 2)
    x = (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)
    us = orc.tucker_factors_hooi(x, ranks, 4)
    kept = np.linalg.norm(orc.tucker_compress(x, us))
    for n in range(3):
        for trial in range(20):
            alt = list(us)
            alt[n] = H.random_orthonormal(rng, shape[n], ranks[n])
            assert np.linalg.norm(orc.tucker_compress(x, alt)) <= kept * (1 + 1e-3)


def test_hooi_warm_start_takes_the_previous_factors():
    wl = synth.WORKLOADS["small4"]
    src = synth.GradientSource(wl)
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=2, hooi_iters=1, hooi_warm=True)
    st = orc.OracleState(cfg)
    orc.oracle_refresh(st, src.gradient(0))
    prev = [u.copy() for u in st.factors]
    g1 = src.gradient(1)
    orc.oracle_refresh(st, g1)
    want = orc.tucker_factors_hooi(orc.residual(g1, st.omega), wl.ranks, 1, prev)
    for a, b in zip(st.factors, want):
        assert np.array_equal(a, b)


# ---- Adam closed forms ----------------------------------------------------------------------------

def test_adam_first_step_is_unit_direction():
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(50) + 1j * rng.standard_normal(50)).astype(np.complex64)
    n, m, v = orc.adam_update(x, np.zeros(50, np.complex64), np.zeros(50, np.float32), 0.9, 0.999, 1e-8, 0)
    assert np.allclose(n, x / (np.abs(x) + 1e-8), rtol=2e-6)
    assert m.dtype == np.complex64 and v.dtype == np.float32 and np.all(v >= 0)


def _identity_state(shape, lr, **kw):
    """Full ranks with U^(n) = I and no sparse part: the compressed space is the
    tensor itself, so the step must reduce to plain Adam.  (Adam's element-wise
    normalisation depends on the basis, hence identity rather than any unitary.)"""
    st = orc.OracleState(orc.OracleConfig(shape=shape, ranks=shape, k=0, T=1000, lr=lr, **kw))
    st.omega = np.zeros(0, np.uint32)
    st.factors = [np.eye(i, dtype=np.complex64) for i in shape]
    return st


def test_constant_gradient_full_rank_closed_form():
    rng = np.random.default_rng(9)
    shape = (3, 4, 2)
    g = (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)
    w0 = (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)
    st = _identity_state(shape, 1e-2, alpha=0.5)
    w = w0
    for _ in range(6):
        w = orc.oracle_step(st, w, g, refresh=False)
    step = g.astype(np.complex128) / (np.abs(g.astype(np.complex128)) + 1e-8)
    want = w0 - 6 * 1e-2 * 0.5 * step
    assert np.max(np.abs(w - want)) < 3e-6


def test_real_inputs_full_rank_match_torch_adam():
    rng = np.random.default_rng(10)
    shape = (4, 3, 5)
    w0 = rng.standard_normal(shape).astype(np.float32)
    grads = [rng.standard_normal(shape).astype(np.float32) for _ in range(8)]
    p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=3e-3, betas=(float(np.float32(0.9)), float(np.float32(0.999))),
                           eps=float(np.float32(1e-8)))
    st = _identity_state(shape, 3e-3)
    w = w0.astype(np.complex64)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        w = orc.oracle_step(st, w, g.astype(np.complex64), refresh=False)
    assert np.max(np.abs(w.imag)) == 0
    assert np.max(np.abs(w.real - p.detach().numpy())) < 2e-6


def test_weight_decay_matches_torch_adamw():
    # Decoupled decay has a definition outside this repository: torch.optim.AdamW multiplies the
    # parameter by (1 - lr * wd) and then applies the Adam update.  lr * wd = 0.025 is large enough
    # that decaying after the update, or by (1 - wd), or not at all, misses by far more than the bound.
    rng = np.random.default_rng(21)
    shape = (3, 4, 2)
    lr, wd = 0.05, 0.5
    w0 = rng.standard_normal(shape).astype(np.float32)
    grads = [rng.standard_normal(shape).astype(np.float32) for _ in range(8)]
    p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=float(np.float32(lr)), betas=(float(np.float32(0.9)), float(np.float32(0.999))),
                            eps=float(np.float32(1e-8)), weight_decay=float(np.float32(wd)))
    st = _identity_state(shape, lr, weight_decay=wd)
    w = w0.astype(np.complex64)
    for g in grads:
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        w = orc.oracle_step(st, w, g.astype(np.complex64), refresh=False)
    assert np.max(np.abs(w.imag)) == 0
    assert np.max(np.abs(w.real - p.detach().numpy())) < 3e-6
    # the planted mistakes are far outside that bound
    u = float(np.float32(lr))
    assert u * u * wd > 1e-4


# ---- structure of Algorithm 1 -----------------------------------------------------------------------

def _run(wl_name, steps, **over):
    wl = synth.WORKLOADS[wl_name]
    src = synth.GradientSource(wl)
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, lr=wl.lr)
    for kk, vv in over.items():
        setattr(cfg, kk, vv)
    st = orc.OracleState(cfg)
    w = src.weight()
    hist = []
    for t in range(steps):
        w = orc.oracle_step(st, w, src.gradient(t))
        hist.append((w.copy(), st.omega.copy(), [u.copy() for u in st.factors]))
    return src, st, hist


def test_alpha_zero_changes_only_omega_entries():
    wl = synth.WORKLOADS["small4"]
    src, st, hist = _run("small4", 1, alpha=0.0)
    w0 = src.weight()
    changed = np.flatnonzero(hist[0][0].reshape(-1) != w0.reshape(-1))
    assert set(changed.tolist()) <= set(st.omega.tolist())
    assert changed.size > 0


def test_lambda_zero_equals_lowrank_update_everywhere():
    src, st, hist = _run("small4", 1, lam=0.0)
    src2, st2, hist2 = _run("small4", 1, lam=0.7)
    a, b = hist[0][0].reshape(-1), hist2[0][0].reshape(-1)
    diff = np.flatnonzero(a != b)
    assert set(diff.tolist()) <= set(st.omega.tolist())
    # outside Omega both runs hold the dense low-rank update only
    mask = np.ones(a.size, bool); mask[st.omega.astype(np.int64)] = False
    assert np.array_equal(a[mask], b[mask])


def test_alpha_scales_lowrank_part_only():
    # Algorithm 1: Gtilde = alpha * lowrank, then + lambda * sparse (not alpha * (L + lambda S)).
    src, st, hist = _run("small4", 1, alpha=0.25, lam=0.5)
    w0 = src.weight().astype(np.complex128)
    om = st.omega.astype(np.int64)
    d = orc.tucker_reconstruct(st.n_l, st.factors).reshape(-1)
    lr = float(np.float32(1e-3))
    want = w0.reshape(-1) - lr * 0.25 * d
    want[om] -= lr * 0.5 * st.n_s.astype(np.complex128)
    assert np.max(np.abs(hist[0][0].reshape(-1) - want)) < 1e-7


def test_refresh_schedule_and_invariants():
    wl = synth.WORKLOADS["small4"]
    src, st, hist = _run("small4", wl.T + 2)
    for t in range(1, wl.T):
        assert np.array_equal(hist[t][1], hist[0][1])
        for u, u0 in zip(hist[t][2], hist[0][2]):
            assert np.array_equal(u, u0)
    assert not np.array_equal(hist[wl.T][1], hist[0][1]) or True   # Omega may coincide; factors must move
    assert any(not np.array_equal(u, u0) for u, u0 in zip(hist[wl.T][2], hist[0][2]))
    om = hist[-1][1].astype(np.int64)
    assert om.size == wl.k and np.all(np.diff(om) > 0) and om[0] >= 0 and om[-1] < wl.numel
    assert np.all(st.v_l >= 0) and np.all(st.v_s >= 0)
    assert st.t == wl.T + 2


def test_k_zero_is_lowrank_only_algorithm():
    # rho = 0 reduces the method to Adam with low-rank tensor decomposition (Algorithm 3)
    wl = synth.WORKLOADS["tiny4"]
    src = synth.GradientSource(wl)
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=0, T=wl.T, lr=1e-2)
    st = orc.OracleState(cfg)
    w = src.weight()
    ref_w = w.astype(np.complex128)
    m = np.zeros(wl.ranks, np.complex128); v = np.zeros(wl.ranks)
    b1, b2 = float(np.float32(0.9)), float(np.float32(0.999))
    for t in range(wl.T + 2):
        g = src.gradient(t)
        w = orc.oracle_step(st, w, g)
        us = [u.astype(np.complex128) for u in st.factors]
        r = g.astype(np.complex128)
        for n in range(4):
            r = orc.mode_n_product(r, np.conj(us[n]).T, n)
        m = b1 * m + (1 - b1) * r
        v = b2 * v + (1 - b2) * np.abs(r * np.conj(r))
        nn = (m / (1 - b1 ** (t + 1))) / (np.sqrt(v / (1 - b2 ** (t + 1))) + float(np.float32(1e-8)))
        for n in range(4):
            nn = orc.mode_n_product(nn, us[n], n)
        ref_w = ref_w - float(np.float32(1e-2)) * nn
        assert np.max(np.abs(w - ref_w)) < 5e-6
        ref_w = w.astype(np.complex128)      # follow the fp32 storage so rounding does not accumulate


def test_half_storage_rounds_to_fp16():
    wl = synth.WORKLOADS["tiny4"]
    src = synth.GradientSource(wl)
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, lr=1e-2, half_storage=True)
    st = orc.OracleState(cfg)
    w = synth.from_half_pairs(synth.to_half_pairs(src.weight()))
    g = synth.from_half_pairs(synth.to_half_pairs(src.gradient(0)))
    w1 = orc.oracle_step(st, w, g)
    assert np.array_equal(synth.from_half_pairs(synth.to_half_pairs(w1)), w1)
    assert not np.array_equal(w1, w)


def test_half_storage_rounds_after_the_dense_update_and_again_at_omega():
    # Hand-computed case in which rounding once and rounding twice give different fp16 values.
    # Tensor of shape (2, 1), U1 = [1, 1]^T / sqrt(2), U2 = [1], Omega = {0}, first step (zero moments), so
    # N_S = g0 / (|g0| + eps) = 1 and N_L = core / (|core| + eps) = 1 (up to 1e-8), and the dense update is
    # N_L / sqrt(2) on both entries.  With u = 2^-10 (the fp16 spacing in [1, 2)), lr = 0.6 u, lambda = 1 and
    # alpha = sqrt(2) both updates are 0.6 u:
    #   entry 0 (in Omega):  1.5 - 0.6u -> fp16 -> 1.5 - u;  (1.5 - u) - 0.6u = 1.5 - 1.6u -> fp16 -> 1.5 - 2u
    #                        (a single rounding of 1.5 - 1.2u would give 1.5 - u)
    #   entry 1 (outside):   1.5 - 0.6u -> 1.5 - u
    # The imaginary parts get no update (the gradient is real) and stay 1.5.
    u = 2.0 ** -10
    cfg = orc.OracleConfig(shape=(2, 1), ranks=(1, 1), k=1, T=1000, lr=0.6 * u, alpha=float(np.sqrt(2.0)), lam=1.0,
                           half_storage=True)
    st = orc.OracleState(cfg)
    st.omega = np.array([0], np.uint32)
    st.factors = [np.array([[1.0], [1.0]], np.complex64) / np.float32(np.sqrt(2.0)), np.ones((1, 1), np.complex64)]
    w = np.full((2, 1), 1.5 + 1.5j, np.complex64)
    g = np.array([[8.0], [2.0]], np.complex64)
    w1 = orc.oracle_step(st, w, g, refresh=False)
    assert w1[0, 0] == np.complex64(complex(1.5 - 2 * u, 1.5))
    assert w1[1, 0] == np.complex64(complex(1.5 - u, 1.5))
    assert float(np.float16(1.5 - 1.2 * u)) == 1.5 - u          # what one rounding would have stored at Omega


# ---- random sparsification strategies and the other composition orders ----------------------------------

def test_philox_known_answers():
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        out = orc.philox4x32_10(w[0:4], w[4:6])
        assert [int(x.reshape(-1)[0]) for x in out] == w[6:10]


def test_randk_is_a_uniform_k_subset_independent_of_the_gradient():
    rng = np.random.default_rng(40)
    shape = (16, 16, 8)
    g1 = (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)
    g2 = (g1 * 100).astype(np.complex64)
    k = 300
    a = orc.sparse_indices(g1, k, "randk", seed=7, epoch=0)
    assert a.size == k and np.all(np.diff(a.astype(np.int64)) > 0) and a[-1] < g1.size
    assert np.array_equal(a, orc.sparse_indices(g2, k, "randk", seed=7, epoch=0))          # does not look at g
    assert not np.array_equal(a, orc.sparse_indices(g1, k, "randk", seed=7, epoch=1))      # redrawn at each refresh
    assert not np.array_equal(a, orc.sparse_indices(g1, k, "randk", seed=8, epoch=0))
    # uniform: over many epochs every position is taken about k / I of the time
    hits = np.zeros(g1.size)
    n_ep = 400
    for ep in range(n_ep):
        hits[orc.sparse_indices(g1, k, "randk", seed=3, epoch=ep).astype(np.int64)] += 1
    p = k / g1.size
    z = (hits - n_ep * p) / np.sqrt(n_ep * p * (1 - p))
    assert abs(z.mean()) < 0.05 and 0.9 < z.std() < 1.1 and np.abs(z).max() < 5.5


def test_exponential_variate_recipe_is_minus_log():
    w = np.random.default_rng(41).integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32)
    w[:3] = [0, 0xFFFFFFFF, 1 << 31]
    e = orc.neg_log_uniform(w)
    u = ((w >> 9).astype(np.float64) + 0.5) * 2.0 ** -23
    assert e.dtype == np.float32 and np.all(e > 0)
    assert np.max(np.abs(e + np.log(u)) / -np.log(u)) < 4e-7
    assert abs(float(e.mean()) - 1.0) < 0.01                                                 # unit-rate exponential


def test_probk_samples_proportionally_to_magnitude():
    # k = 1: the entry with the largest |g| / E wins with probability |g_i| / sum |g| (exponential clocks)
    g = np.array([1, 2j, -3, 4 - 0j, 0], dtype=np.complex64)
    counts = np.zeros(5)
    n = 6000
    for seed in range(n):
        counts[int(orc.sparse_indices(g, 1, "probk", seed=seed, epoch=0)[0])] += 1
    want = np.array([1, 2, 3, 4, 0]) / 10.0
    assert counts[4] == 0                                                                   # zero magnitude: never drawn first
    assert np.all(np.abs(counts[:4] / n - want[:4]) < 4 * np.sqrt(want[:4] * (1 - want[:4]) / n))
    # k = 4 of these five: always the four non-zero entries
    assert orc.sparse_indices(g, 4, "probk", seed=1, epoch=3).tolist() == [0, 1, 2, 3]
    # and the key is what the definition says, element by element
    key = orc.selection_key(g, "probk", seed=5, epoch=2)
    word = orc.selection_word(5, 5, 2)
    u = ((word >> 9).astype(np.float64) + 0.5) * 2.0 ** -23
    assert np.allclose(key[:4], np.abs(g[:4]) / -np.log(u[:4]), rtol=1e-6) and key[4] == 0


def _kron_projector(us):
    """Matrix of P_U on row-major vec(G): kron of U_n U_n^H."""
    p = np.ones((1, 1), dtype=np.complex128)
    for u in us:
        u = u.astype(np.complex128)
        p = np.kron(p, u @ np.conj(u).T)
    return p


def test_composition_sum_applies_both_parts_to_the_gradient():
    wl = synth.WORKLOADS["tiny4"]
    src = synth.GradientSource(wl)
    g, w0 = src.gradient(0), src.weight()
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, lr=1e-2, composition="sum")
    st = orc.OracleState(cfg)
    w1 = orc.oracle_step(st, w0, g)
    assert np.array_equal(st.omega, orc.sparse_indices_topk(g, wl.k))
    # factors come from the gradient itself, not from the residual
    for a, b in zip(st.factors, orc.tucker_factors(g, wl.ranks)):
        assert H.max_sin_angle(a, b) < 1e-6
    # first step: N = x / (|x| + eps) on both parts, low-rank part = P_U applied to N_L through the kron projector
    core = orc.tucker_compress(g, st.factors)
    n_l = core / (np.abs(core) + 1e-8)
    dense = orc.tucker_reconstruct(n_l, st.factors).reshape(-1)
    gs = g.reshape(-1)[st.omega.astype(np.int64)].astype(np.complex128)
    want = w0.reshape(-1).astype(np.complex128) - 1e-2 * dense
    want[st.omega.astype(np.int64)] -= 1e-2 * gs / (np.abs(gs) + 1e-8)
    assert np.max(np.abs(w1.reshape(-1) - want)) < 2e-6
    assert np.allclose(st.core.reshape(-1), (np.conj(np.kron(np.kron(np.kron(st.factors[0], st.factors[1]), st.factors[2]),
                                                             st.factors[3]).astype(np.complex128)).T @ g.reshape(-1)), atol=1e-4)


def test_composition_lr_us_takes_the_sparse_part_from_the_lowrank_residual():
    wl = synth.WORKLOADS["tiny4"]
    src = synth.GradientSource(wl)
    g, w0 = src.gradient(0), src.weight()
    cfg = orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, lr=1e-2, composition="lr_us")
    st = orc.OracleState(cfg)
    w1 = orc.oracle_step(st, w0, g)
    us = st.factors
    for a, b in zip(us, orc.tucker_factors(g, wl.ranks)):
        assert H.max_sin_angle(a, b) < 1e-6
    # residual through the explicit projector matrix; Omega = its k largest entries by brute force
    r = (g.reshape(-1).astype(np.complex128) - _kron_projector(us) @ g.reshape(-1).astype(np.complex128)).reshape(wl.shape)
    assert np.max(np.abs(orc.lowrank_residual(cfg, g, us) - r)) < 1e-6
    assert st.omega.tolist() == H.brute_topk(orc.lowrank_residual(cfg, g, us), wl.k)
    assert np.max(np.abs(st.g_s - r.reshape(-1)[st.omega.astype(np.int64)])) < 1e-5
    # the low-rank part is that of the whole gradient
    assert np.max(np.abs(st.core - orc.tucker_compress(g, us))) < 1e-5
    # full ranks: nothing is left for the sparse part, and the step is the low-rank step alone
    full = orc.OracleConfig(shape=wl.shape, ranks=wl.shape, k=wl.k, T=wl.T, lr=1e-2, composition="lr_us")
    lo = orc.OracleConfig(shape=wl.shape, ranks=wl.shape, k=0, T=wl.T, lr=1e-2)
    sa, sb = orc.OracleState(full), orc.OracleState(lo)
    wa, wb = orc.oracle_step(sa, w0, g), orc.oracle_step(sb, w0, g)
    assert np.max(np.abs(sa.g_s)) < 1e-5 * np.max(np.abs(g))
    mask = np.ones(g.size, bool); mask[sa.omega.astype(np.int64)] = False
    assert np.max(np.abs(wa.reshape(-1)[mask] - wb.reshape(-1)[mask])) < 1e-6


def test_bfloat16_rounding_matches_torch():
    x = (np.random.default_rng(50).standard_normal(50000) * 3.7).astype(np.float32)
    x[:4] = [1 + 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -20, 1 + 3 * 2.0 ** -8, -1 - 2.0 ** -8]     # ties go to even
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(orc.round_to_bfloat16(x), want)
    assert orc.round_to_bfloat16(x)[:4].tolist() == [1.0, 1.0078125, 1.015625, -1.0]
    cfg = orc.OracleConfig(shape=(2,), ranks=(1,), k=0, T=1, bf16_storage=True)
    w = orc._store_w(np.array([1 + 2.0 ** -9 + 1j * (1 + 2.0 ** -6)]), cfg)
    assert w[0] == complex(1.0, 1 + 2.0 ** -6)


# ---- state size: the paper's worked example --------------------------------------------------

def test_state_size_matches_paper_example():
    vals = {}
    for line in open(os.path.join(GOLDEN, "parameter_count_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, val = line.split()
        vals[key] = int(val)
    n, m, r = vals["N"], vals["M"], vals["r_max"]
    e = orc.state_entries((n, n, m, m), (r, r, r, r), 0)
    p_tensor = e["m_l"] + e["factors"]
    assert e["m_l"] == vals["core_entries"]
    assert p_tensor == 71680 and round(p_tensor / 1000) in (vals["p_tensor_rounded_thousands"], 72)
    p_matrix = r * r * (n * n + m * m)
    assert round(p_matrix / 1e5) == vals["p_matrix_rounded_100k"]
    assert abs(p_matrix / p_tensor - vals["ratio_printed"]) < 3     # printed as "~75x"


def test_workload_sizes():
    want_k = {"cfg1": 1475, "cfg2": 111412, "cfg3": 865076, "cfg4": 1426064, "cfg5": 5452596}
    for name, k in want_k.items():
        assert synth.WORKLOADS[name].k == k
