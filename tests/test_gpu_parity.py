"""GPU-vs-oracle parity through the C ABI (run with -m gpu on a B200)."""
import numpy as np
import pytest
import torch

from oracle import tgrad_oracle as orc
from paper_2501_02379_b200 import binding as B
from paper_2501_02379_b200 import synth
from tests import helpers as H
from tests.parity import Pair, to_device, from_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny4", "small4", "small5", "ragged4", "small3", "odd4", "odd32", "small5b",
                                  "half65", "lead200", "lead300", "tail19", "gram144", "gram96h", "gram75"])
def test_trajectory_small(name):
    wl = synth.WORKLOADS[name]
    p = Pair(wl)
    for t in range(wl.steps):
        p.step(t)
    print(name, p.report)


def test_matrix_case():
    # N = 2: the Tucker factors are the singular subspaces of the matrix (the oracle's N = 2 case is pinned to
    # numpy.linalg.svd).  On a refresh step the core is diagonal up to rounding, hence the stage-wise weight check.
    wl = synth.WORKLOADS["mat2"]
    p = Pair(wl, stagewise_w=True)
    for t in range(wl.steps):
        p.step(t)
    assert p.gst.shape == wl.shape and len(p.gst.factors()) == 2
    print("mat2", p.report)


def test_trajectory_cfg1_full():
    wl = synth.WORKLOADS["cfg1"]
    p = Pair(wl)
    for t in range(wl.steps):
        p.step(t)
    print("cfg1", p.report)


@pytest.mark.parametrize("name", ["small4", "ragged4", "odd32", "cfg1"])
def test_trajectory_warm_refresh(name):
    # every refresh after the first starts the eigensolver from the previous eigenvectors: same subspaces, same
    # orthonormality, same trajectory tolerances
    wl = synth.WORKLOADS[name]
    p = Pair(wl, warm_refresh=True)
    for t in range(max(wl.steps, 3 * wl.T + 1)):
        p.step(t)
    print(name, p.report)


@pytest.mark.parametrize("name,warm", [("small4", False), ("ragged4", False), ("odd32", True), ("cfg1", True), ("small5", False)])
def test_hooi_refinement(name, warm):
    # TuckerFactors with two refinement sweeps (higher-order orthogonal iteration) on noisier gradients, where the
    # refined subspaces differ visibly from the truncated-SVD ones; warm: later refreshes start from the stored
    # factors and skip the truncated-SVD stage
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS[name], noise_scale=0.1)
    p = Pair(wl, warm_refresh=warm, hooi_iters=2)
    for t in range(2 * wl.T + 1):
        p.step(t)
    g = p.src.gradient(0)
    res = orc.residual(g, orc.sparse_indices_topk(g, wl.k))
    plain, refined = orc.tucker_factors(res, wl.ranks), orc.tucker_factors_hooi(res, wl.ranks, 2)
    moved = max(H.max_sin_angle(a, b) for a, b in zip(plain, refined))
    assert moved > 5e-3, f"the refinement barely moves the subspaces here ({moved}): the test would not notice its absence"
    print("hooi", name, p.report.get("angle"), "moved", moved)


@pytest.mark.parametrize("name", ["small4", "ragged4", "odd32"])
@pytest.mark.parametrize("strategy", ["randk", "probk"])
def test_random_sparsification_strategies(name, strategy):
    # Omega from one Philox word per entry (uniform k-subset) or from |g| / exponential variate (sampling proportional
    # to |g|): the same bits on both sides, so the sets are compared exactly, and they change from refresh to refresh
    wl = synth.WORKLOADS[name]
    p = Pair(wl, strategy=strategy, seed=0x1234567890ABCDEF)
    sets = []
    for t in range(2 * wl.T + 1):
        p.step(t)
        if t % wl.T == 0:
            sets.append(p.gst.export(B.WHAT_OMEGA))
    assert not np.array_equal(sets[0], sets[1]) and not np.array_equal(sets[1], sets[2])
    if strategy == "randk":
        assert not np.array_equal(sets[0], orc.sparse_indices_topk(p.src.gradient(0), wl.k))


@pytest.mark.parametrize("name,half", [("small4", False), ("odd32", False), ("ragged4", True), ("small5b", False), ("mat2", False)])
@pytest.mark.parametrize("composition", ["sum", "lr_us"])
def test_other_compositions(name, half, composition):
    # "sum": both parts see the gradient itself; "lr_us": the low-rank part goes first and the sparse part is chosen
    # from, and fed with, G - P_U(G)
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS[name], half_storage=half)
    p = Pair(wl, composition=composition, stagewise_w=(name == "mat2"))
    for t in range(wl.T + 2):
        p.step(t)
    print(composition, name, p.report.get("omega_boundary_entries"), p.report.get("core"), p.report.get("m_s"))


def test_alpha_lambda_weight_decay():
    wl = synth.WORKLOADS["small4"]
    p = Pair(wl, alpha=0.25, lam=0.5, weight_decay=0.1, lr=1e-2)
    for t in range(wl.T + 2):
        p.step(t)


def test_k_zero_lowrank_only():
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS["small4"], rho=(0, 1), outlier_frac=(0, 1))
    assert wl.k == 0
    p = Pair(wl)
    for t in range(wl.T + 1):
        p.step(t)


def test_k_equals_numel_sparse_only():
    # every entry is selected: the residual, its Gram matrices and the core are zero, any orthonormal U^(n) is a valid
    # factor (so the subspaces are not compared), and the update is the sparse branch alone
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS["small4"], rho=(1, 1), outlier_frac=(0, 1))
    assert wl.k == wl.numel
    p = Pair(wl)
    g = p.src.gradient(0)
    p.gst.refresh_subspace(to_device(g, False))
    orc.oracle_refresh(p.ost, g)
    assert p.gst.query_status()[0] == 0
    assert np.array_equal(p.gst.export(B.WHAT_OMEGA), np.arange(wl.numel, dtype=np.uint32))
    us = p.gst.factors()
    for u in us:
        assert H.ortho_defect(u) <= 1e-5
    p.ost.factors = [u.copy() for u in us]
    for t in range(3):
        g = p.src.gradient(t)
        p.gst.step(p.w_dev, to_device(g, False))
        p.w_ref = orc.oracle_step(p.ost, p.w_ref, g, refresh=False)
        p.compare()
    assert not np.any(p.gst.export(B.WHAT_CORE))


def test_topk_ties_bit_exact():
    # tie-heavy quantised gradients, all-equal magnitudes, k in {1, I-1, I}
    shape = (12, 10, 8, 5)
    n = int(np.prod(shape))
    for seed, k in [(0, 137), (1, 1), (2, n - 1), (3, n), (4, 2048), (5, 2049)]:
        g = synth.quantised_ties(shape, 3, seed)
        cfg = B.make_config(shape, (4, 3, 3, 2), k, 4, auto_refresh=False)
        st = B.TgradState(cfg)
        st.refresh_subspace(to_device(g, False))
        assert np.array_equal(st.export(B.WHAT_OMEGA), orc.sparse_indices_topk(g, k)), (seed, k)
    g = np.full(shape, 1 - 2j, dtype=np.complex64)
    cfg = B.make_config(shape, (4, 3, 3, 2), 777, 4, auto_refresh=False)
    st = B.TgradState(cfg)
    st.refresh_subspace(to_device(g, False))
    assert np.array_equal(st.export(B.WHAT_OMEGA), np.arange(777, dtype=np.uint32))


def test_topk_multi_block_ragged():
    # several compaction blocks plus a ragged tail, ties across block borders
    shape = (37, 11, 9, 7)
    g = synth.quantised_ties(shape, 40, 11)
    n = g.size
    for k in (1, 5000, n // 2):
        cfg = B.make_config(shape, (4, 3, 3, 2), k, 4, auto_refresh=False)
        st = B.TgradState(cfg)
        st.refresh_subspace(to_device(g, False))
        assert np.array_equal(st.export(B.WHAT_OMEGA), orc.sparse_indices_topk(g, k)), k


@pytest.mark.parametrize("name", ["ragged4", "odd32", "odd4", "small3"])
def test_half_storage_small(name):
    # fp16-stored W and G: the general kernels (24-row slabs) and the fp16-MMA kernels (8k / 16k-row slabs)
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS[name], half_storage=True)
    p = Pair(wl)
    for t in range(wl.T + 2):
        p.step(t)
    print("half", name, p.report)


@pytest.mark.parametrize("name", ["ragged4", "odd32", "small3", "gram96h"])
def test_bf16_storage_small(name):
    # bfloat16-stored W and G (the other reading of the mixed recipe's "half precision"): general kernels
    import dataclasses
    wl = dataclasses.replace(synth.WORKLOADS[name], bf16_storage=True, half_storage=False)
    p = Pair(wl)
    for t in range(wl.T + 2):
        p.step(t)
    print("bf16", name, p.report)


@pytest.mark.parametrize("composition", ["us_lr", "sum"])
def test_diagnostics_against_the_definitions(composition):
    wl = synth.WORKLOADS["ragged4"]
    p = Pair(wl, composition=composition)
    p.step(0)
    g = p.src.gradient(1)
    g_dev = to_device(g, False)
    p.step(1)
    gn, share, lost, defect = p.gst.diagnostics(g_dev)
    g128 = g.astype(np.complex128)
    us = p.ost.factors
    gs = g128.reshape(-1)[p.ost.omega.astype(np.int64)]
    x = orc.residual(g, p.ost.omega).astype(np.complex128) if composition == "us_lr" else g128
    want_lost = np.linalg.norm(x - orc.tucker_reconstruct(orc.tucker_compress(x, us), us)) / np.linalg.norm(g128)
    assert abs(gn - np.linalg.norm(g128)) <= 1e-6 * gn
    assert abs(share - np.linalg.norm(gs) / np.linalg.norm(g128)) <= 1e-6
    assert abs(lost - want_lost) <= 1e-4 * max(want_lost, 1e-3)
    assert abs(defect - max(H.ortho_defect(u) for u in us)) <= 2e-7 and defect < 1e-5


def test_auto_refresh_matches_explicit():
    wl = synth.WORKLOADS["small4"]
    src = synth.GradientSource(wl)
    outs = []
    for auto in (True, False):
        cfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=auto)
        st = B.TgradState(cfg)
        w = to_device(src.weight(), False)
        for t in range(wl.T + 2):
            g = to_device(src.gradient(t), False)
            if not auto and t % wl.T == 0:
                st.refresh_subspace(g)
            st.step(w, g)
        outs.append((from_device(w, False), st.export(B.WHAT_M_L), st.export(B.WHAT_OMEGA)))
    for a, b in zip(outs[0], outs[1]):
        assert np.array_equal(a, b)


def test_export_import_resume_bitwise():
    wl = synth.WORKLOADS["small4"]
    src = synth.GradientSource(wl)
    total = 2 * wl.T + 3
    cut = wl.T + 1
    cfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T)
    a = B.TgradState(cfg)
    wa = to_device(src.weight(), False)
    snap = None
    for t in range(total):
        if t == cut:
            snap = {w: a.export(w) for w in (B.WHAT_OMEGA, B.WHAT_M_L, B.WHAT_V_L, B.WHAT_M_S, B.WHAT_V_S)}
            snap["factors"] = a.factors()
            snap["w"] = wa.clone()
        a.step(wa, to_device(src.gradient(t), False))
    b = B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T))
    for w in (B.WHAT_OMEGA, B.WHAT_M_L, B.WHAT_V_L, B.WHAT_M_S, B.WHAT_V_S):
        b.import_(w, snap[w])
    for n, u in enumerate(snap["factors"]):
        b.import_(B.WHAT_FACTOR_BASE + n, u)
    b.set_step(cut)
    wb = snap["w"]
    for t in range(cut, total):
        b.step(wb, to_device(src.gradient(t), False))
    assert torch.equal(wa, wb)
    for w in (B.WHAT_OMEGA, B.WHAT_M_L, B.WHAT_V_L, B.WHAT_M_S, B.WHAT_V_S):
        assert np.array_equal(a.export(w), b.export(w))
    assert a.query_status()[1] == b.query_status()[1] == total


def test_factors_imported_mid_run_take_effect():
    # a state that has already stepped (so every table derived from the factors exists) gets new factors through the
    # C ABI; its next step must equal, bit for bit, that of a fresh state given the same factors from the start
    wl = synth.WORKLOADS["odd32"]                # 32 x 17 slabs: the tensor-core streaming kernels
    src = synth.GradientSource(wl)
    cfg = B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False)
    a = B.TgradState(cfg)
    wa = to_device(src.weight(), False)
    a.refresh_subspace(to_device(src.gradient(0), False))
    for t in range(2):
        a.step(wa, to_device(src.gradient(t), False))
    rng = np.random.default_rng(5)
    new_u = [H.random_orthonormal(rng, i, r).astype(np.complex64) for i, r in zip(wl.shape, wl.ranks)]
    for n, u in enumerate(new_u):
        a.import_(B.WHAT_FACTOR_BASE + n, u)
    b = B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False))
    for w in (B.WHAT_OMEGA, B.WHAT_M_L, B.WHAT_V_L, B.WHAT_M_S, B.WHAT_V_S):
        b.import_(w, a.export(w))
    for n, u in enumerate(new_u):
        b.import_(B.WHAT_FACTOR_BASE + n, u)
    b.set_step(2)
    wb = wa.clone()
    g = src.gradient(2)
    a.step(wa, to_device(g, False))
    b.step(wb, to_device(g, False))
    assert torch.equal(wa, wb)
    for w in (B.WHAT_M_L, B.WHAT_V_L, B.WHAT_CORE):
        assert np.array_equal(a.export(w), b.export(w))


def test_batched_matches_single():
    wl = synth.WORKLOADS["small4"]
    srcs = [synth.GradientSource(wl, i) for i in range(3)]
    single, batched = [], []
    for mode in ("single", "batched"):
        sts = [B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T)) for _ in srcs]
        ws = [to_device(s.weight(), False) for s in srcs]
        for t in range(wl.T + 1):
            gs = [to_device(s.gradient(t), False) for s in srcs]
            if mode == "single":
                for st, w, g in zip(sts, ws, gs):
                    st.step(w, g)
            else:
                B.step_batched(sts, ws, gs)
        (single if mode == "single" else batched).extend(ws)
    for a, b in zip(single, batched):
        assert torch.equal(a, b)


@pytest.mark.parametrize("name", ["ragged4", "gram75"])
def test_batched_refresh_matches_single(name):
    # five tensors (more than the library has side streams) refreshed one by one and through the batched call: the same
    # index sets and factors, bit for bit, and the gradients left as they were
    wl = synth.WORKLOADS[name]
    gs = [synth.GradientSource(wl, i).gradient(0) for i in range(5)]
    out = {}
    for mode in ("single", "batched"):
        sts = [B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False)) for _ in gs]
        gd = [to_device(g, False) for g in gs]
        if mode == "single":
            for st, g in zip(sts, gd):
                st.refresh_subspace(g)
        else:
            B.refresh_subspace_batched(sts, gd)
        torch.cuda.synchronize()
        out[mode] = [(st.export(B.WHAT_OMEGA), st.factors()) for st in sts]
        for st in sts:
            assert st.query_status()[0] == 0
        for g, d in zip(gs, gd):
            assert np.array_equal(from_device(d, False), g)
    for (oa, fa), (ob, fb) in zip(out["single"], out["batched"]):
        assert np.array_equal(oa, ob)
        for ua, ub in zip(fa, fb):
            assert np.array_equal(ua, ub)


def test_nonfinite_sets_flag():
    wl = synth.WORKLOADS["small4"]
    g = synth.GradientSource(wl).gradient(0)
    g.reshape(-1)[5] = np.nan
    st = B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False))
    st.refresh_subspace(to_device(g, False))
    flags, _, _ = st.query_status()
    assert flags & B.FLAG_NONFINITE


def test_warm_refresh_recovers_from_a_nonfinite_gradient():
    # a refresh on a gradient with a NaN leaves a useless eigenvector basis behind; the next warm-started refresh must
    # notice and start from the identity, so that its factors are those of the new (finite) gradient
    wl = synth.WORKLOADS["ragged4"]
    src = synth.GradientSource(wl)
    st = B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False, warm_refresh=True))
    st.refresh_subspace(to_device(src.gradient(0), False))
    g = src.gradient(1).copy()
    g.reshape(-1)[7] = np.nan
    st.refresh_subspace(to_device(g, False))
    assert st.query_status()[0] & B.FLAG_NONFINITE
    g2 = src.gradient(2)
    st.refresh_subspace(to_device(g2, False))
    ost = orc.OracleState(orc.OracleConfig(shape=wl.shape, ranks=wl.ranks, k=wl.k, T=wl.T, half_storage=False, lr=1e-3,
                                           alpha=1.0, lam=1.0, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0))
    orc.oracle_refresh(ost, g2)
    assert np.array_equal(st.export(B.WHAT_OMEGA), ost.omega)
    for ug, uo in zip(st.factors(), ost.factors):
        assert np.all(np.isfinite(ug))
        assert H.max_sin_angle(ug, uo) <= 1e-3
        assert H.ortho_defect(ug) <= 1e-5


def test_jacobi_cap_sets_flag_not_hang():
    wl = synth.WORKLOADS["small4"]
    g = synth.GradientSource(wl).gradient(0)
    st = B.TgradState(B.make_config(wl.shape, wl.ranks, wl.k, wl.T, auto_refresh=False, jacobi_max_sweeps=1,
                                    jacobi_tol=1e-12))
    st.refresh_subspace(to_device(g, False))
    flags, _, sweeps = st.query_status()
    assert flags & B.FLAG_NO_CONVERGE and max(sweeps) == 1
