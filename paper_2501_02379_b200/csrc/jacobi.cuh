// Cyclic Jacobi eigensolver for the small Hermitian PSD Gram matrices A_n, and
// extraction of the factor matrices U^(n): eigenvectors of the r_n largest
// eigenvalues in descending order, each scaled by the unit phase that makes its
// largest-modulus component real and positive.
//
// One thread block per mode.  Rotations of one stage of a round-robin ordering
// act on disjoint index pairs, so a stage is: (1) rotation angles for all pairs,
// (2) column update of A and V, (3) row update of A.  Every loop is bounded by
// the sweep cap; reaching the cap sets a sticky flag instead of spinning.
#pragma once
#include "common.cuh"

namespace tg {

constexpr int JAC_MAX_N = 1024;
constexpr int JAC_THREADS = 1024;

struct JacobiMode {
  cf* A;        // n x n, row-major, overwritten (diagonalised)
  cf* V;        // n x n scratch (accumulated rotations)
  cf* U;        // out: n x r row-major
  int n, r;
};
struct JacobiParams {
  JacobiMode mode[8];
  int max_sweeps;
  float tol;
  int* flags;   // flags[0] sticky bits, flags[1 + mode] sweeps used
};

struct JacRot { float c, s, gx, gy, npp, nqq; int p, q; };

__global__ void __launch_bounds__(JAC_THREADS) jacobi_kernel(JacobiParams P) {
  const JacobiMode md = P.mode[blockIdx.x];
  const int n = md.n, r = md.r;
  cf* __restrict__ A = md.A;
  cf* __restrict__ V = md.V;
  __shared__ JacRot rot[JAC_MAX_N / 2];
  __shared__ float red[32];
  __shared__ int nrot;
  __shared__ float lam[JAC_MAX_N];
  __shared__ int rank_of[JAC_MAX_N];
  const int tid = threadIdx.x, nt = blockDim.x;

  for (int i = tid; i < n * n; i += nt) { int a = i / n, b = i - a * n; V[i] = make_float2(a == b ? 1.f : 0.f, 0.f); }
  // scale of the matrix: largest diagonal entry
  float dmax = 0.f;
  for (int i = tid; i < n; i += nt) dmax = fmaxf(dmax, fabsf(A[(size_t)i * n + i].x));
  for (int o = 16; o; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
  if ((tid & 31) == 0) red[tid >> 5] = dmax;
  __syncthreads();
  dmax = 0.f;
  for (int w = 0; w < (nt >> 5); ++w) dmax = fmaxf(dmax, red[w]);
  const float thr2 = (P.tol * dmax) * (P.tol * dmax);

  const int m = (n + 1) & ~1;       // even number of players (one phantom if n is odd)
  const int half = m >> 1;
  int sweep = 0;
  bool converged = (n < 2);
  for (; sweep < P.max_sweeps && !converged; ++sweep) {
    int rotated_this_sweep = 0;
    for (int stage = 0; stage < m - 1; ++stage) {
      if (tid == 0) nrot = 0;
      __syncthreads();
      // (1) rotation parameters
      if (tid < half) {
        int p, q;
        if (tid == 0) { p = m - 1; q = stage; }
        else { p = (stage + tid) % (m - 1); q = (stage - tid + (m - 1)) % (m - 1); }
        if (p > q) { int t = p; p = q; q = t; }
        JacRot R; R.p = p; R.q = q; R.c = 1.f; R.s = 0.f; R.gx = 1.f; R.gy = 0.f; R.npp = 0.f; R.nqq = 0.f;
        if (q < n) {
          float a = A[(size_t)p * n + p].x, d = A[(size_t)q * n + q].x;
          cf b = A[(size_t)p * n + q];
          float b2 = b.x * b.x + b.y * b.y;
          if (b2 > thr2 && b2 > 0.f) {
            // angle in double: c^2 + s^2 = 1 to fp32 rounding, so V stays orthonormal over thousands of rotations
            double abd = sqrt((double)b.x * b.x + (double)b.y * b.y);
            double tau = ((double)d - (double)a) / (2.0 * abd);
            double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
            double cd = 1.0 / sqrt(1.0 + t * t);
            R.c = (float)cd; R.s = (float)(t * cd);
            R.gx = (float)(b.x / abd); R.gy = (float)(-b.y / abd);   // g = exp(-i phi) = conj(b)/|b|
            R.npp = (float)(a - t * abd); R.nqq = (float)(d + t * abd);
            atomicAdd(&nrot, 1);
          } else {
            R.p = -1;                                  // nothing to do for this pair
          }
        } else {
          R.p = -1;
        }
        rot[tid] = R;
      }
      __syncthreads();
      const int applied = nrot;
      rotated_this_sweep += applied;
      if (applied) {
        // (2) X <- X J on the columns (p, q) of A and V:  x_p' = c x_p - s g x_q,  x_q' = s x_p + c g x_q
        for (int task = tid; task < 2 * n * half; task += nt) {
          int pr = task % half; int rest = task / half; int i = rest % n; int which = rest / n;
          JacRot R = rot[pr];
          if (R.p < 0) continue;
          cf* X = which ? V : A;
          cf xp = X[(size_t)i * n + R.p], xq = X[(size_t)i * n + R.q];
          cf gq = make_float2(R.gx * xq.x - R.gy * xq.y, R.gx * xq.y + R.gy * xq.x);
          X[(size_t)i * n + R.p] = make_float2(R.c * xp.x - R.s * gq.x, R.c * xp.y - R.s * gq.y);
          X[(size_t)i * n + R.q] = make_float2(R.s * xp.x + R.c * gq.x, R.s * xp.y + R.c * gq.y);
        }
        __syncthreads();
        // (3) A <- J^H A on the rows (p, q):  r_p' = c r_p - s conj(g) r_q,  r_q' = s r_p + c conj(g) r_q
        for (int task = tid; task < n * half; task += nt) {
          int j = task % n, pr = task / n;
          JacRot R = rot[pr];
          if (R.p < 0) continue;
          cf xp = A[(size_t)R.p * n + j], xq = A[(size_t)R.q * n + j];
          cf gq = make_float2(R.gx * xq.x + R.gy * xq.y, R.gx * xq.y - R.gy * xq.x);
          cf np_ = make_float2(R.c * xp.x - R.s * gq.x, R.c * xp.y - R.s * gq.y);
          cf nq_ = make_float2(R.s * xp.x + R.c * gq.x, R.s * xp.y + R.c * gq.y);
          if (j == R.p) { np_ = make_float2(R.npp, 0.f); nq_ = make_float2(0.f, 0.f); }
          if (j == R.q) { np_ = make_float2(0.f, 0.f); nq_ = make_float2(R.nqq, 0.f); }
          A[(size_t)R.p * n + j] = np_;
          A[(size_t)R.q * n + j] = nq_;
        }
      }
      __syncthreads();
    }
    converged = (rotated_this_sweep == 0);
  }
  if (tid == 0) {
    P.flags[1 + blockIdx.x] = sweep;
    if (!converged) atomicOr(&P.flags[0], 1);
  }
  // eigenvalues, descending rank (ties: lower index first)
  for (int i = tid; i < n; i += nt) lam[i] = A[(size_t)i * n + i].x;
  __syncthreads();
  for (int i = tid; i < n; i += nt) {
    float li = lam[i]; int rk = 0;
    for (int j = 0; j < n; ++j) { float lj = lam[j]; rk += (lj > li) || (lj == li && j < i); }
    rank_of[i] = rk;
  }
  __syncthreads();
  // one warp per kept eigenvector: canonical phase, write U[:, rank]
  const int warp = tid >> 5, lane = tid & 31, nwarps = nt >> 5;
  for (int i = warp; i < n; i += nwarps) {
    int rk = rank_of[i];
    if (rk >= r) continue;
    float best = -1.f; int bi = 0;
    for (int a = lane; a < n; a += 32) {
      cf v = V[(size_t)a * n + i];
      float mg = v.x * v.x + v.y * v.y;
      if (mg > best) { best = mg; bi = a; }
    }
    for (int o = 16; o; o >>= 1) {
      float ob = __shfl_xor_sync(0xffffffffu, best, o);
      int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    cf pv = V[(size_t)bi * n + i];
    float mg = sqrtf(pv.x * pv.x + pv.y * pv.y);
    cf ph = mg > 0.f ? make_float2(pv.x / mg, -pv.y / mg) : make_float2(1.f, 0.f);
    for (int a = lane; a < n; a += 32) {
      cf v = V[(size_t)a * n + i];
      md.U[(size_t)a * r + rk] = make_float2(v.x * ph.x - v.y * ph.y, v.x * ph.y + v.y * ph.x);
    }
  }
}

}  // namespace tg
