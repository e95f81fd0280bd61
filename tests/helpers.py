"""Shared test utilities: comparison metrics and brute-force references.

Nothing here implements the optimizer; these are measuring sticks.
"""
import numpy as np


FLOOR_FRAC = 2.0 ** -7            # every workload with a full oracle comparison passes at 2^-8 or tighter (most at 2^-16)
FLOOR_FRAC_LARGE = 2.0 ** -5      # the 545 M-entry configuration, whose 2 M-entry core comes from fp16-stored operands


def rel_err(a, b, floor_frac=FLOOR_FRAC):
    """max_i |a_i - b_i| / max(|b_i|, tau), tau = floor_frac * rms(b).

    Every entry of a compressed tensor is a sum of the same number of terms of the
    same typical size, so fp32 arithmetic (unit roundoff u = 2^-24) leaves an
    absolute error of a few u * rms(b) on each entry whatever its own size: the
    intermediate tensors of the chain are stored in fp32 (u * rms each), and each
    partial sum rounds.  Measured: rms error 2-4 u, maximum over 1e4..2e6 entries
    up to about 20 u.  An entry much smaller than rms(b) is the result of
    cancellation and cannot carry a 1e-4 *relative* accuracy in fp32; the bound
    1e-4 * tau (13 u * rms at the default floor 2^-7, 52 u * rms at 2^-5) is the absolute
    accuracy asked of those entries, and every entry above tau must meet 1e-4 relative
    to itself.
    """
    a = np.asarray(a).reshape(-1).astype(np.complex128)
    b = np.asarray(b).reshape(-1).astype(np.complex128)
    if b.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(np.abs(b) ** 2))
    tau = floor_frac * rms
    den = np.maximum(np.abs(b), tau if tau > 0 else 1.0)
    return float(np.max(np.abs(a - b) / den))


FLOOR_CONTRACT = 1e-3


def below_floor_fraction(b, floor_frac=FLOOR_CONTRACT):
    """Share of the reference entries smaller than tau = floor_frac * rms(b)."""
    b = np.asarray(b).reshape(-1).astype(np.complex128)
    if b.size == 0:
        return 0.0
    rms = np.sqrt(np.mean(np.abs(b) ** 2))
    return float(np.mean(np.abs(b) < floor_frac * rms))


def tightest_floor_log2(a, b, tol=1e-4, lo=5, hi=16):
    """Largest j in [lo, hi] such that rel_err(a, b, 2^-j) <= tol (the error is monotone in the floor);
    lo - 1 if even 2^-lo fails."""
    best = lo - 1
    for j in range(lo, hi + 1):
        if rel_err(a, b, 2.0 ** -j) <= tol:
            best = j
        else:
            break
    return best


def fro_err(a, b):
    a = np.asarray(a).reshape(-1).astype(np.complex128)
    b = np.asarray(b).reshape(-1).astype(np.complex128)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (nb if nb > 0 else 1.0))


def max_sin_angle(u, v):
    """Largest principal-angle sine between span(u) and span(v) (both with
    orthonormal columns): || (I - v v^H) u ||_2."""
    u = np.asarray(u, dtype=np.complex128)
    v = np.asarray(v, dtype=np.complex128)
    resid = u - v @ (np.conj(v).T @ u)
    return float(np.linalg.norm(resid, 2))


def ortho_defect(u):
    u = np.asarray(u, dtype=np.complex128)
    return float(np.max(np.abs(np.conj(u).T @ u - np.eye(u.shape[1]))))


def brute_topk(g, k):
    """Pure-Python top-k: sort all (key, index) pairs, key descending then
    index ascending; key = fp32 re*re + im*im with separately rounded ops."""
    flat = np.asarray(g).reshape(-1)
    pairs = []
    for i in range(flat.size):
        re = np.float32(flat[i].real)
        im = np.float32(flat[i].imag)
        key = np.float32(np.float32(re * re) + np.float32(im * im))
        pairs.append((-float(key), i))
    pairs.sort()
    return sorted(i for _, i in pairs[:k])


def random_orthonormal(rng, n, r):
    a = rng.standard_normal((n, r)) + 1j * rng.standard_normal((n, r))
    q, _ = np.linalg.qr(a)
    return q
