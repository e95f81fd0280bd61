"""CPU oracle for the TensorGRaD optimizer step (Algorithm 1 of the paper).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of
what the paper defines.  It shares no code with the CUDA library, is never
imported by it, and must only be used by the tests, the smoke check and the
benchmark's CPU-baseline leg.

Every function names the passage it follows.  Contractions run in complex128,
stored optimizer states are rounded to fp32 once per step (the paper keeps the
optimizer states in full precision, Section 2.3), the top-k key is computed in
fp32 exactly as the selection rule fixes it.

Conventions where the paper is silent (each one is a stated reading, not a
fact of the paper -- "parity unpinned" against the authors' own code for
these): beta1/beta2/eps values, alpha on the low-rank part only (the
reconstruction steps of Algorithm 1, not the equation of Section 2.2), bias correction with t+1,
moments carried over unchanged across refreshes (slot-wise for the sparse
ones), decoupled weight decay, fp16 storage of W/G in the mixed recipe.

Sign convention: the caller passes grad = d(phi)/dW; Algorithm 1 defines
G = -grad and W <- W + eta * Gtilde(G).  Every stage is odd in the sign of G
(or even, for V), so the oracle evaluates the stages on grad and subtracts.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------
# Sparse part (Section 2.2, "Unstructured sparse gradient tensor")
# --------------------------------------------------------------------------

def magnitude_key(g: np.ndarray) -> np.ndarray:
    """|g|^2 as fp32: fl(fl(re*re) + fl(im*im)), no fused multiply-add.

    Top-k *magnitude* selection orders entries by |g|; squaring is monotone,
    and this fp32 expression is the precision in which the decision is taken.
    numpy rounds each float32 operation separately.
    """
    g = np.asarray(g)
    re = np.ascontiguousarray(g.real, dtype=np.float32)
    im = np.ascontiguousarray(g.imag, dtype=np.float32)
    return (re * re) + (im * im)


def sparse_indices_topk(g: np.ndarray, k: int) -> np.ndarray:
    """SparseIndices(G, rho, top-k) of Algorithm 1, with k = ceil(rho I).

    The k entries largest under (key descending, flat row-major index
    ascending); returned as ascending flat indices (uint32).  A stable sort of
    the negated key keeps equal keys in index order.
    """
    key = magnitude_key(g).reshape(-1)
    if k < 0 or k > key.size:
        raise ValueError("k out of range")
    order = np.argsort(-key, kind="stable")
    return np.sort(order[:k]).astype(np.uint32)


# ---- the other two sparsification strategies of Section 2.2 ("probabilistic sampling, or uniform random
#      selection"); the paper names them without defining them, so the definitions below are stated readings ----

_PHILOX_M0, _PHILOX_M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter, key):
    """Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
    SC 2011): counter = four uint32 arrays (or scalars), key = two uint32 scalars; returns four uint32 arrays.
    Round: (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)); the key is bumped by
    the Weyl constants (W0, W1) between rounds."""
    c = [np.asarray(x, dtype=np.uint64) & np.uint64(0xFFFFFFFF) for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = int(key[0]) & 0xFFFFFFFF, int(key[1]) & 0xFFFFFFFF
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = _PHILOX_M0 * c[0]
        p1 = _PHILOX_M1 * c[2]
        c = [(p1 >> np.uint64(32)) ^ c[1] ^ np.uint64(k0), p1 & mask, (p0 >> np.uint64(32)) ^ c[3] ^ np.uint64(k1), p0 & mask]
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return [x.astype(np.uint32) for x in c]


def selection_word(numel: int, seed: int, epoch: int) -> np.ndarray:
    """One 32-bit random word per flat index i for the refresh number `epoch`: the first output word of
    Philox-4x32-10 with counter (i, epoch, 0, 0) and key (seed mod 2^32, seed div 2^32)."""
    i = np.arange(numel, dtype=np.uint64)
    return philox4x32_10((i, np.uint64(epoch), np.uint64(0), np.uint64(0)), (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))[0]


_LN2_F = np.float32(0.693147182)
_SQRT2_F = np.float32(1.41421354)
_C3, _C5, _C7, _C9 = np.float32(1.0 / 3.0), np.float32(0.2), np.float32(1.0 / 7.0), np.float32(1.0 / 9.0)


def neg_log_uniform(word: np.ndarray) -> np.ndarray:
    """E = -ln(u), u = ((word >> 9) + 1/2) 2^-23 in (0, 1), evaluated in fp32 by a fixed sequence of IEEE operations
    (no fused multiply-add) so that every implementation gets the same bits: u = m 2^e with m in (sqrt(1/2), sqrt(2)],
    f = m - 1, s = f / (f + 2), z = s s, ln m = 2 (s + s z (1/3 + z (1/5 + z (1/7 + z / 9)))), ln u = e ln 2 + ln m.
    An exponential variate of unit rate up to the 1e-7 relative error of the series."""
    w = np.asarray(word, dtype=np.uint32)
    u = ((w >> np.uint32(9)).astype(np.float32) + np.float32(0.5)) * np.float32(2.0 ** -23)
    bits = u.view(np.uint32)
    e = (bits >> np.uint32(23)).astype(np.int32) - 127
    m = ((bits & np.uint32(0x7FFFFF)) | np.uint32(0x3F800000)).view(np.float32)
    big = m > _SQRT2_F
    m = np.where(big, m * np.float32(0.5), m).astype(np.float32)
    e = np.where(big, e + 1, e)
    f = m - np.float32(1.0)
    s_ = f / (f + np.float32(2.0))
    z = s_ * s_
    p = _C9 * z
    p = p + _C7
    p = p * z
    p = p + _C5
    p = p * z
    p = p + _C3
    r = s_ * z
    r = r * p
    r = r + s_
    r = r * np.float32(2.0)
    ln_u = e.astype(np.float32) * _LN2_F
    ln_u = ln_u + r
    return (-ln_u).astype(np.float32)


def selection_key(g: np.ndarray, strategy: str, seed: int = 0, epoch: int = 0) -> np.ndarray:
    """The non-negative fp32 key whose k largest values (ties to the lower flat index) define Omega.
    topk:  |g|^2 (magnitude_key).
    randk: the random word itself, as an integer: a uniformly random k-subset, independent of g.
    probk: |g| / E with E a unit-rate exponential variate per entry -- the k largest of these are a sample of k
           entries without replacement with probabilities proportional to |g| (the exponential-clocks form of
           weighted reservoir sampling, Efraimidis and Spirakis 2006); |g| = sqrt of the fp32 key, division in fp32."""
    if strategy == "topk":
        return magnitude_key(g).reshape(-1)
    word = selection_word(int(np.asarray(g).size), seed, epoch)
    if strategy == "randk":
        return word
    if strategy == "probk":
        w = np.sqrt(magnitude_key(g).reshape(-1))
        return (w / neg_log_uniform(word)).astype(np.float32)
    raise ValueError(strategy)


def sparse_indices(g: np.ndarray, k: int, strategy: str = "topk", seed: int = 0, epoch: int = 0) -> np.ndarray:
    """SparseIndices(G, rho, strategy) of Algorithm 1: the k entries with the largest selection_key, ties to the
    lower flat index, as ascending flat indices."""
    if strategy == "topk":
        return sparse_indices_topk(g, k)
    key = selection_key(g, strategy, seed, epoch)
    if k < 0 or k > key.size:
        raise ValueError("k out of range")
    bits = key.view(np.uint32) if key.dtype == np.float32 else key
    order = np.argsort(-(bits.astype(np.int64)), kind="stable")
    return np.sort(order[:k]).astype(np.uint32)


def sparse_gather(g: np.ndarray, omega: np.ndarray) -> np.ndarray:
    """Sparse(G, Omega): the values at the stored indices (the per-step
    "create sparse tensor" statement of Algorithm 1)."""
    return np.asarray(g).reshape(-1)[omega.astype(np.int64)].copy()


def residual(g: np.ndarray, omega: np.ndarray) -> np.ndarray:
    """R = G - Sparse(G, Omega): G with the entries at Omega set to zero
    (Section 2.2 "Residual and composition"; the subtraction inside Algorithm 1)."""
    r = np.array(g, copy=True, order="C")
    r.reshape(-1)[omega.astype(np.int64)] = 0      # C-contiguous: reshape is a view
    return r


# --------------------------------------------------------------------------
# Tensor algebra (Appendix "Tensor Operations and Notation")
# --------------------------------------------------------------------------

def unfold(x: np.ndarray, n: int) -> np.ndarray:
    """Mode-n unfolding: mode-n fibres as columns, remaining indices ordered
    first-index-fastest (Definition "Mode-k Unfolding")."""
    return np.reshape(np.moveaxis(x, n, 0), (x.shape[n], -1), order="F")


def mode_n_product(x: np.ndarray, u: np.ndarray, n: int) -> np.ndarray:
    """(X x_n U)[.., j, ..] = sum_{i_n} X[.., i_n, ..] U[j, i_n]
    (Definition "Mode-k Product"; U is J x I_n)."""
    y = np.tensordot(u, x, axes=([1], [n]))      # new index j first
    return np.moveaxis(y, 0, n)


def tucker_compress(r: np.ndarray, factors: Sequence[np.ndarray]) -> np.ndarray:
    """G_L = R x_1 U1^H ... x_N UN^H  (Section 2.2 low-rank compression,
    the "low-rank compression" statement of Algorithm 1; complex tensors take conjugate transposes, Remark
    "Real-Valued Analysis").  Modes are contracted in the order written."""
    x = np.asarray(r, dtype=np.complex128)
    for n, u in enumerate(factors):
        x = mode_n_product(x, np.conj(np.asarray(u, dtype=np.complex128)).T, n)
    return x


def tucker_reconstruct(c: np.ndarray, factors: Sequence[np.ndarray]) -> np.ndarray:
    """Gtilde_L = C x_1 U1 ... x_N UN (Section 2.2; the "reconstruct low-rank
    part" statement of Algorithm 1)."""
    x = np.asarray(c, dtype=np.complex128)
    for n, u in enumerate(factors):
        x = mode_n_product(x, np.asarray(u, dtype=np.complex128), n)
    return x


def mode_gram(r: np.ndarray, n: int) -> np.ndarray:
    """A_n = R_(n) R_(n)^H (Hermitian PSD, I_n x I_n), complex128."""
    m = unfold(np.asarray(r, dtype=np.complex128), n)
    return m @ np.conj(m).T


def canonical_phase(u: np.ndarray) -> np.ndarray:
    """Multiply each column by the unit phase that makes its largest-modulus
    component real and positive (first such row on ties)."""
    u = np.array(u, copy=True)
    for j in range(u.shape[1]):
        col = u[:, j]
        i = int(np.argmax(np.abs(col)))
        a = col[i]
        if a != 0:
            u[:, j] = col * (np.conj(a) / np.abs(a))
    return u


def tucker_factors(r: np.ndarray, ranks: Sequence[int]) -> List[np.ndarray]:
    """TuckerFactors(R, r) of Algorithm 1.

    Each U^(n) holds the r_n leading left singular vectors of the mode-n
    unfolding of R (the truncated-SVD stage of the decomposition described in
    Appendix "Tensor Decomposition / Implementation"), obtained here as the
    eigenvectors of the r_n largest eigenvalues of A_n = R_(n) R_(n)^H, in
    descending eigenvalue order, phase-canonicalised, stored as complex64.
    No refinement iterations are applied.
    """
    out = []
    for n, rn in enumerate(ranks):
        a = mode_gram(r, n)
        w, v = np.linalg.eigh(a)                      # ascending eigenvalues
        v = v[:, ::-1][:, :rn]
        out.append(np.ascontiguousarray(canonical_phase(v).astype(np.complex64)))
    return out


def tucker_factors_hooi(r: np.ndarray, ranks: Sequence[int], n_iter: int,
                        init: Optional[Sequence[np.ndarray]] = None) -> List[np.ndarray]:
    """TuckerFactors(R, r) with the refinement the paper's implementation applies (Appendix "Tensor Decomposition /
    Implementation": factors from truncated SVDs of the mode-n unfoldings, then refined iteratively to reduce the
    Frobenius reconstruction error, optionally restarted from previous factors).

    Higher-order orthogonal iteration: starting from `init` (the truncated-SVD factors of tucker_factors when None),
    each of the n_iter sweeps visits the modes in order and replaces U^(n) by the r_n leading left singular vectors
    of the mode-n unfolding of  Y = R x_{m != n} U^(m)H  (every other mode compressed with its current factor, the
    factors already updated in this sweep included), obtained as eigenvectors of Y_(n) Y_(n)^H, descending,
    phase-canonicalised, stored as complex64.  n_iter = 0 returns the starting factors.
    """
    us = [np.asarray(u, dtype=np.complex64) for u in (init if init is not None else tucker_factors(r, ranks))]
    x = np.asarray(r, dtype=np.complex128)
    for _ in range(int(n_iter)):
        for n, rn in enumerate(ranks):
            y = x
            for m, u in enumerate(us):
                if m != n:
                    y = mode_n_product(y, np.conj(u.astype(np.complex128)).T, m)
            w, v = np.linalg.eigh(mode_gram(y, n))
            us[n] = np.ascontiguousarray(canonical_phase(v[:, ::-1][:, :rn]).astype(np.complex64))
    return us


# --------------------------------------------------------------------------
# Adam in the compressed space (AdamUpdate of Algorithm 1; UPDATE block of Algorithm 3)
# --------------------------------------------------------------------------

def adam_update(x, m, v, beta1, beta2, eps, t):
    """One Adam update of a compressed gradient x (complex) with first moment m
    (complex64) and second moment v (float32).  Returns (N, m_new, v_new):

        M <- b1 M + (1-b1) x          V <- b2 V + (1-b2) |x conj(x)|
        N  = (M / (1-b1^(t+1))) / (sqrt(V / (1-b2^(t+1))) + eps)

    t is the 0-based step counter, so the correction uses t+1.  The corrected
    moments are temporaries: the stored ones are the un-corrected M and V,
    rounded to fp32.
    """
    b1 = float(np.float32(beta1)); b2 = float(np.float32(beta2)); e = float(np.float32(eps))
    x = np.asarray(x, dtype=np.complex128)
    m_new = (b1 * np.asarray(m, dtype=np.complex128) + (1.0 - b1) * x).astype(np.complex64)
    v_new = (b2 * np.asarray(v, dtype=np.float64)
             + (1.0 - b2) * (x.real * x.real + x.imag * x.imag)).astype(np.float32)
    n = adam_direction(m_new, v_new, beta1, beta2, eps, t)
    return n, m_new, v_new


def adam_direction(m, v, beta1, beta2, eps, t):
    """N = (M / (1-b1^(t+1))) / (sqrt(V / (1-b2^(t+1))) + eps): the bias-corrected,
    normalised update computed from stored (un-corrected) moments (last three
    statements of the UPDATE block of Algorithm 3)."""
    b1 = float(np.float32(beta1)); b2 = float(np.float32(beta2)); e = float(np.float32(eps))
    c1 = float(np.float32(1.0 - b1 ** (t + 1)))
    c2 = float(np.float32(1.0 - b2 ** (t + 1)))
    return (np.asarray(m, dtype=np.complex128) / c1) / (np.sqrt(np.asarray(v, dtype=np.float64) / c2) + e)


# --------------------------------------------------------------------------
# The step (Algorithm 1)
# --------------------------------------------------------------------------

@dataclasses.dataclass
class OracleConfig:
    shape: Sequence[int]
    ranks: Sequence[int]
    k: int
    T: int
    lr: float = 1e-3
    alpha: float = 1.0
    lam: float = 1.0
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    weight_decay: float = 0.0
    half_storage: bool = False      # W and G live as fp16 (re, im) pairs
    bf16_storage: bool = False      # ... or as bfloat16 pairs (the paper's recipe says "half precision" without naming the format)
    hooi_iters: int = 0             # refinement sweeps of TuckerFactors (0: truncated-SVD factors only)
    hooi_warm: bool = False         # refinement starts from the factors of the previous refresh when there are any
    strategy: str = "topk"          # topk | randk | probk (Section 2.2, sparsification strategies)
    seed: int = 0                   # of the random strategies
    composition: str = "us_lr"      # us_lr: Algorithm 1 (sparse first, low rank on the residual);
                                    # lr_us: low rank first, sparse part taken from G - P_U(G);
                                    # sum: both applied to the gradient itself and added (Section 2.2 "Residual and
                                    # composition"; the combination ablation)


def round_to_bfloat16(x: np.ndarray) -> np.ndarray:
    """float32 values rounded to bfloat16 (8 exponent bits, 7 explicit mantissa bits), nearest, ties to even,
    returned as float32: the upper 16 bits of the fp32 pattern after adding half a unit of the last kept place
    (one less on an even keeper)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    bias = ((u >> np.uint64(16)) & np.uint64(1)) + np.uint64(0x7FFF)
    r = ((u + bias) & np.uint64(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32).reshape(np.shape(x))


def _store_w(w: np.ndarray, half, bf16: bool = False) -> np.ndarray:
    """Round a complex128 weight to its storage type and widen it back.  `half` may be the configuration."""
    if isinstance(half, OracleConfig):
        half, bf16 = half.half_storage, half.bf16_storage
    if bf16:
        re = round_to_bfloat16(w.real.astype(np.float32)).astype(np.float64)
        im = round_to_bfloat16(w.imag.astype(np.float32)).astype(np.float64)
        return re + 1j * im
    if half:
        re = w.real.astype(np.float16).astype(np.float64)
        im = w.imag.astype(np.float16).astype(np.float64)
        return re + 1j * im
    return w.astype(np.complex64).astype(np.complex128)


class OracleState:
    """State of Algorithm 1 for one weight tensor (its initialisation statements)."""

    def __init__(self, cfg: OracleConfig):
        self.cfg = cfg
        self.t = 0
        p = tuple(int(r) for r in cfg.ranks)
        self.omega: Optional[np.ndarray] = None
        self.factors: Optional[List[np.ndarray]] = None
        self.m_l = np.zeros(p, dtype=np.complex64)
        self.v_l = np.zeros(p, dtype=np.float32)
        self.m_s = np.zeros(cfg.k, dtype=np.complex64)
        self.v_s = np.zeros(cfg.k, dtype=np.float32)
        # last step's intermediates, kept for inspection by tests
        self.core = None
        self.n_l = None
        self.g_s = None
        self.n_s = None


def _factors_of(cfg: OracleConfig, x: np.ndarray, prev) -> List[np.ndarray]:
    if cfg.hooi_iters > 0:
        init = prev if (cfg.hooi_warm and prev is not None) else None
        return tucker_factors_hooi(x, cfg.ranks, cfg.hooi_iters, init)
    return tucker_factors(x, cfg.ranks)


def lowrank_residual(cfg: OracleConfig, grad: np.ndarray, factors) -> np.ndarray:
    """G - P_U(G), P_U(G) = (G x_n U^(n)H) x_n U^(n), rounded to the storage type of the gradient: what the sparse
    part sees when the low-rank part goes first."""
    x = np.asarray(grad, dtype=np.complex128)
    return _store_w(x - tucker_reconstruct(tucker_compress(x, factors), factors), cfg).astype(np.complex64)


def oracle_refresh(st: OracleState, grad: np.ndarray) -> None:
    """The `t mod T = 0` branch of Algorithm 1: new Omega, residual, new factors.  Moments are
    left untouched (nothing in the loop resets them).  The first component sees the gradient, the second the
    residual of the first (composition "sum": both see the gradient)."""
    cfg = st.cfg
    epoch = st.t // cfg.T
    if cfg.composition == "us_lr":
        st.omega = sparse_indices(grad, cfg.k, cfg.strategy, cfg.seed, epoch)
        st.factors = _factors_of(cfg, residual(grad, st.omega), st.factors)
    elif cfg.composition == "sum":
        st.omega = sparse_indices(grad, cfg.k, cfg.strategy, cfg.seed, epoch)
        st.factors = _factors_of(cfg, np.asarray(grad), st.factors)
    elif cfg.composition == "lr_us":
        st.factors = _factors_of(cfg, np.asarray(grad), st.factors)
        st.omega = sparse_indices(lowrank_residual(cfg, grad, st.factors), cfg.k, cfg.strategy, cfg.seed, epoch)
    else:
        raise ValueError(cfg.composition)


def weight_update(cfg: OracleConfig, w: np.ndarray, n_l: np.ndarray, n_s: np.ndarray, omega: np.ndarray,
                  factors: Sequence[np.ndarray]) -> np.ndarray:
    """The last statements of the loop body of Algorithm 1 ("reconstruct low-rank part", "add scaled sparse
    tensor", "update weights"), signs flipped as the module docstring says:

        W <- (1 - eta wd) W;  W <- W - eta alpha (N_L x_1 U1 ... x_N UN);  W[Omega] <- W[Omega] - eta lambda N_S

    with one rounding to the storage type after the dense update and one more, at Omega, after the sparse add."""
    lr = float(np.float32(cfg.lr)); al = float(np.float32(cfg.alpha)); la = float(np.float32(cfg.lam))
    wd = float(np.float32(cfg.weight_decay))
    wn = np.asarray(w, dtype=np.complex128)
    if wd != 0.0:
        wn = wn * (1.0 - lr * wd)
    d = tucker_reconstruct(n_l, factors)
    wn = np.ascontiguousarray(_store_w(wn - (lr * al) * d, cfg))
    flat = wn.reshape(-1)                          # a view of the contiguous array
    om = np.asarray(omega).astype(np.int64)
    flat[om] = _store_w(flat[om] - (lr * la) * np.asarray(n_s, dtype=np.complex128), cfg)
    return wn.astype(np.complex64)


def oracle_step(st: OracleState, w: np.ndarray, grad: np.ndarray, refresh: Optional[bool] = None) -> np.ndarray:
    """One pass of the loop body of Algorithm 1 for one tensor.

    w, grad: complex arrays of cfg.shape holding values exactly representable
    in the storage type.  Returns the new weight (complex64, or complex64
    holding fp16-representable values for half storage).
    refresh=None follows the schedule t mod T = 0; True/False overrides it.
    """
    cfg = st.cfg
    do_refresh = (st.t % cfg.T == 0) if refresh is None else refresh
    if do_refresh:
        oracle_refresh(st, grad)
    # sparse values, residual, low-rank compression
    if cfg.composition == "us_lr":
        g_s = sparse_gather(grad, st.omega).astype(np.complex64)
        core = tucker_compress(residual(grad, st.omega), st.factors).astype(np.complex64)
    elif cfg.composition == "sum":
        g_s = sparse_gather(grad, st.omega).astype(np.complex64)
        core = tucker_compress(grad, st.factors).astype(np.complex64)
    else:
        # low rank first: the core of the gradient itself; the sparse values are those of G - P_U(G), with P_U(G)
        # rebuilt from the core as stored (fp32)
        core = tucker_compress(grad, st.factors).astype(np.complex64)
        low = tucker_reconstruct(core, st.factors).reshape(-1)[st.omega.astype(np.int64)]
        g_s = (sparse_gather(grad, st.omega).astype(np.complex128) - low).astype(np.complex64)
    # AdamUpdate on both compressed parts
    n_s, st.m_s, st.v_s = adam_update(g_s, st.m_s, st.v_s, cfg.beta1, cfg.beta2, cfg.eps, st.t)
    n_l, st.m_l, st.v_l = adam_update(core, st.m_l, st.v_l, cfg.beta1, cfg.beta2, cfg.eps, st.t)
    n_s = n_s.astype(np.complex64); n_l = n_l.astype(np.complex64)
    wn = weight_update(cfg, w, n_l, n_s, st.omega, st.factors)
    st.core, st.n_l, st.g_s, st.n_s = core, n_l, g_s, n_s
    st.t += 1
    return wn


def state_entries(shape, ranks, k):
    """Optimizer-state entry counts (Appendix "Parameter Complexity Analysis"):
    core-shaped moments, factor matrices, sparse indices and sparse moments."""
    p = int(np.prod(ranks, dtype=np.int64))
    fac = int(sum(int(i) * int(r) for i, r in zip(shape, ranks)))
    return {"m_l": p, "v_l": p, "factors": fac, "omega": int(k), "m_s": int(k), "v_s": int(k)}
