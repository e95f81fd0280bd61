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
  int index[8];     // tensor mode each entry belongs to
  int max_sweeps;
  float tol;
  int* flags;   // flags[0] sticky bits, flags[1 + mode] sweeps used, flags[JAC_SKIP + mode] != 0: nothing to do
};

// A mode whose factor matrix this refresh has already been produced (by the subspace iteration) is skipped by every
// kernel of this file.
constexpr int JAC_SKIP = 16;

struct JacRot { float c, s, gx, gy, npp, nqq; int p, q; };

__global__ void __launch_bounds__(JAC_THREADS) jacobi_kernel(JacobiParams P) {
  const JacobiMode md = P.mode[blockIdx.x];
  if (P.flags[JAC_SKIP + P.index[blockIdx.x]]) return;
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
    P.flags[1 + P.index[blockIdx.x]] = sweep;
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

// ---------------------------------------------------------------------------------------------
// Fast path for n <= JAC_SMEM_MAX_N: the matrix lives in shared memory, and the accumulation of
// the eigenvectors is taken off the critical path.
//
// (1) jacobi_sweeps_kernel, one block per mode: the same round-robin ordering and the same
//     rotations as above, applied to A alone.  With the index set split into the n/2 disjoint
//     pairs of a stage, A <- J^H A J is an independent update of every 2 x 2 block
//     A[{p_I, q_I}][{p_J, q_J}] by the rotations of pairs I and J, so a stage is: rotation
//     parameters, barrier, all blocks, barrier.  Every rotation is appended to a log in global
//     memory: (c, s, g.x, g.y), identity when the pair needed none.
// (2) jacobi_vectors_kernel, one warp per row of V: starting from the unit vector e_i, replays
//     the log on its row (V <- V J acts on rows independently), then stores the row.
// (3) jacobi_factors_kernel, one block per mode: eigenvalue ranks, canonical phase, U.
// ---------------------------------------------------------------------------------------------
constexpr int JAC_SMEM_MAX_N = 160;      // 160^2 complex64 = 200 KB of shared memory
constexpr int JAC_FAST_MAX_N = 256;      // up to here the same kernel runs with the matrix in global memory (L2)

struct JacobiFastMode {
  const cf* A;       // n x n input (left untouched)
  cf* work;          // n x (n | 1) working copy in global memory, used when n > JAC_SMEM_MAX_N
  float4* log;       // [sweeps][m-1][m/2] rotations
  float* lam;        // out: n eigenvalues (unsorted)
  cf* V;             // out: n x n eigenvectors in columns (row-major)
  cf* U;             // out: n x r
  int n, r;
  int index;         // tensor mode this entry belongs to
  int row0;          // first global warp index of this mode's rows in jacobi_vectors_kernel
};
struct JacobiFastParams {
  JacobiFastMode mode[8];
  int nmodes, total_rows;
  int row_stride;    // jacobi_vectors_kernel: complex entries per warp row buffer (>= largest n)
  int max_sweeps;
  float tol;
  int* flags;        // flags[0] sticky bits, flags[1 + mode] sweeps used, flags[JAC_SKIP + mode]
};

// the pair of players (p < q) that meet at table `tb` in stage `stage` of a round robin of m players
__host__ __device__ inline size_t jac_log_entries(int n, int max_sweeps) {
  const size_t m = (size_t)((n + 1) & ~1);
  return (size_t)max_sweeps * (m - 1) * (m / 2);
}
__host__ __device__ inline size_t jac_a_bytes(int n) { return ((size_t)n * (n | 1) * sizeof(cf) + 15) & ~(size_t)15; }
__host__ __device__ inline size_t jac_sweeps_smem(int n, bool insmem = true) {
  const size_t m = (size_t)((n + 1) & ~1);
  return (insmem ? jac_a_bytes(n) : 0) + (m / 2) * (sizeof(float4) + sizeof(float2) + sizeof(int2));
}

__device__ __forceinline__ void jac_pair(int m, int stage, int tb, int& p, int& q) {
  if (tb == 0) { p = m - 1; q = stage; }
  else {
    p = stage + tb; if (p >= m - 1) p -= m - 1;        // stage < m-1 and tb < m/2: one wrap at most
    q = stage - tb; if (q < 0) q += m - 1;
  }
  if (p > q) { int t = p; p = q; q = t; }
}

// One Newton step of (x, y) towards x^2 + y^2 = 1.  The defect e = 1 - x^2 - y^2 is formed without
// rounding (products split into rounded part and exact remainder; the two subtractions are exact
// because x^2 + y^2 is already within a few ulp of 1), so the step leaves only the unbiased final
// rounding of x and y: the accumulated eigenvectors then lose orthonormality like a random walk.
__device__ __forceinline__ void jac_unit(float& x, float& y) {
  const float p = x * x, ep = fmaf(x, x, -p), q = y * y, eq = fmaf(y, y, -q);
  const float hi = fmaxf(p, q), lo = fminf(p, q);
  const float e = ((1.f - hi) - lo) - (ep + eq);
  x = fmaf(0.5f * e, x, x); y = fmaf(0.5f * e, y, y);
}

// Rotation that annihilates the (p, q) entry b of the Hermitian 2 x 2 block [[a, b], [conj(b), d]], in fp32.
// c and s (and the phase g = conj(b)/|b|) get one Newton step towards c^2 + s^2 = 1 (|g| = 1): what keeps the
// accumulated eigenvectors orthonormal over thousands of rotations is that normalisation, not the angle.
__device__ __forceinline__ void jac_rotation(float a, float d, cf b, float absb, JacRot& R) {
  const float tau = (d - a) / (2.f * absb);
  const float t = copysignf(1.f, tau) / (fabsf(tau) + sqrtf(fmaf(tau, tau, 1.f)));
  float c = rsqrtf(fmaf(t, t, 1.f)), s = t * c;
  jac_unit(c, s);
  const float inv = 1.f / absb;
  float gx = b.x * inv, gy = -b.y * inv;
  jac_unit(gx, gy);
  R.c = c; R.s = s; R.gx = gx; R.gy = gy;
  R.npp = a - t * absb; R.nqq = d + t * absb;
}

// The same with the hardware's approximate reciprocal, square root and reciprocal square root (each good to a
// few ulp, but several times shorter than the IEEE sequences): the angle is then off by a few ulp, which the next
// sweep sees as a slightly larger remainder, while c^2 + s^2 = 1 and |g| = 1 are restored by jac_unit as above.
// On the critical path of every stage of the rotation-log kernels, where all other warps wait for these values.
__device__ __forceinline__ void jac_rotation_fast(float a, float d, cf b, float b2, JacRot& R) {
  const float inv = rsqrtf(b2), absb = b2 * inv;
  const float tau = 0.5f * (d - a) * inv, at = fminf(fabsf(tau), 1e18f);     // the cap keeps tau^2 finite
  const float q = fmaf(at, at, 1.f);
  const float t = copysignf(__fdividef(1.f, at + q * rsqrtf(q)), tau);
  float c = rsqrtf(fmaf(t, t, 1.f)), s = t * c;
  jac_unit(c, s);
  float gx = b.x * inv, gy = -b.y * inv;
  jac_unit(gx, gy);
  R.c = c; R.s = s; R.gx = gx; R.gy = gy;
  R.npp = a - t * absb; R.nqq = d + t * absb;
}

// Only the upper triangle of A (i <= j) is kept up to date: A is Hermitian before and after every
// stage, so block (I, J) with I < J determines block (J, I), and half of the shared-memory traffic
// -- which is what bounds this kernel -- goes away.
__device__ __forceinline__ cf jac_get(const cf* A, int ld, int i, int j) {
  if (i <= j) return A[(size_t)i * ld + j];
  cf v = A[(size_t)j * ld + i];
  return make_float2(v.x, -v.y);
}
__device__ __forceinline__ void jac_put(cf* A, int ld, int i, int j, cf v) {
  if (i <= j) A[(size_t)i * ld + j] = v;
  else A[(size_t)j * ld + i] = make_float2(v.x, -v.y);
}

// INSMEM: the matrix is in shared memory (n <= JAC_SMEM_MAX_N); otherwise in the mode's global work buffer, where
// a block's own writes are visible to it after a barrier.
template <bool INSMEM>
__global__ void __launch_bounds__(JAC_THREADS) jacobi_sweeps_kernel(JacobiFastParams P) {
  extern __shared__ __align__(16) unsigned char jsm[];
  const JacobiFastMode md = P.mode[blockIdx.x];
  if (P.flags[JAC_SKIP + md.index]) return;
  const int n = md.n;
  const int m = (n + 1) & ~1, half = m >> 1;
  cf* A = INSMEM ? reinterpret_cast<cf*>(jsm) : md.work;               // [n][n | 1], upper triangle live
  float4* rotc = reinterpret_cast<float4*>(jsm + (INSMEM ? jac_a_bytes(n) : 0));      // [half] (c, s, g.x, g.y); 16-byte aligned
  float2* rotd = reinterpret_cast<float2*>(rotc + half);               // [half] new diagonal entries of the pair
  int2* rotp = reinterpret_cast<int2*>(rotd + half);                   // [half] (p, q); p < 0: no rotation, p = -1 - p
  __shared__ float red[32];
  const int tid = threadIdx.x, nt = blockDim.x;
  const int ld = n | 1;      // odd row stride: column accesses (the mirrored half) spread over the banks
  const cf* Ain = md.A;
  for (int i = tid; i < n * n; i += nt) { const int r_ = i / n, c_ = i - r_ * n; A[(size_t)r_ * ld + c_] = Ain[i]; }
  __syncthreads();
  float dmax = 0.f;
  for (int i = tid; i < n; i += nt) dmax = fmaxf(dmax, fabsf(A[(size_t)i * ld + i].x));
  for (int o = 16; o; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
  if ((tid & 31) == 0) red[tid >> 5] = dmax;
  __syncthreads();
  dmax = 0.f;
  for (int w = 0; w < (nt >> 5); ++w) dmax = fmaxf(dmax, red[w]);
  const float thr2 = (P.tol * dmax) * (P.tol * dmax);

  // The blocks (I <= J) of the upper triangle are spread evenly: with he = half rounded up to even, cell
  // (r, c), r < he/2, stands for block (r, c) if r <= c and for block (he-1-r, he-1-c) otherwise; the
  // cells r == c also take the diagonal block he-1-r.  Pair indices >= half do not exist.
  const int he = (half + 1) & ~1, R = he >> 1;
  const int rpp = nt / he;                      // rows of cells per pass
  const int cc = tid % he, I0 = tid / he;
  const bool worker = tid < rpp * he;
  // B <- J_I^H B J_J for the 2 x 2 block of pairs (I, J), I <= J
  auto do_block = [&](int I, int J) {
    if (J >= half) return;
    const int2 pqI = rotp[I], pqJ = rotp[J];
    if (pqI.x < 0 && pqJ.x < 0) return;
    const int pJ = pqJ.x < 0 ? -1 - pqJ.x : pqJ.x, qJ = pqJ.y;
    if (I == J) {                                // the rotated pair itself: exactly diagonal
      const float2 dd = rotd[I];
      A[(size_t)pJ * ld + pJ] = make_float2(dd.x, 0.f);
      A[(size_t)qJ * ld + qJ] = make_float2(dd.y, 0.f);
      A[(size_t)pJ * ld + qJ] = make_float2(0.f, 0.f);
      return;
    }
    const float4 cI = rotc[I], cJ = rotc[J];
    const int pI = pqI.x < 0 ? -1 - pqI.x : pqI.x, qI = pqI.y;
    const bool qIok = qI < n, qJok = qJ < n;
    // where the four entries live in the upper triangle (32-bit offsets), and whether they are stored conjugated
    const bool s00 = pI > pJ, s01 = pI > qJ, s10 = qI > pJ, s11 = qI > qJ;
    const int i00 = s00 ? pJ * ld + pI : pI * ld + pJ, i01 = s01 ? qJ * ld + pI : pI * ld + qJ;
    const int i10 = s10 ? pJ * ld + qI : qI * ld + pJ, i11 = s11 ? qJ * ld + qI : qI * ld + qJ;
    const cf z = make_float2(0.f, 0.f);
    cf x00 = A[i00], x01 = qJok ? A[i01] : z, x10 = qIok ? A[i10] : z, x11 = (qIok && qJok) ? A[i11] : z;
    if (s00) x00.y = -x00.y;
    if (s01) x01.y = -x01.y;
    if (s10) x10.y = -x10.y;
    if (s11) x11.y = -x11.y;
    // columns: x_p' = c x_p - s g x_q,  x_q' = s x_p + c g x_q
    {
      cf g0 = make_float2(cJ.z * x01.x - cJ.w * x01.y, cJ.z * x01.y + cJ.w * x01.x);
      cf g1 = make_float2(cJ.z * x11.x - cJ.w * x11.y, cJ.z * x11.y + cJ.w * x11.x);
      cf y00 = make_float2(cJ.x * x00.x - cJ.y * g0.x, cJ.x * x00.y - cJ.y * g0.y);
      cf y01 = make_float2(cJ.y * x00.x + cJ.x * g0.x, cJ.y * x00.y + cJ.x * g0.y);
      cf y10 = make_float2(cJ.x * x10.x - cJ.y * g1.x, cJ.x * x10.y - cJ.y * g1.y);
      cf y11 = make_float2(cJ.y * x10.x + cJ.x * g1.x, cJ.y * x10.y + cJ.x * g1.y);
      x00 = y00; x01 = y01; x10 = y10; x11 = y11;
    }
    // rows: r_p' = c r_p - s conj(g) r_q,  r_q' = s r_p + c conj(g) r_q
    {
      cf g0 = make_float2(cI.z * x10.x + cI.w * x10.y, cI.z * x10.y - cI.w * x10.x);
      cf g1 = make_float2(cI.z * x11.x + cI.w * x11.y, cI.z * x11.y - cI.w * x11.x);
      cf y00 = make_float2(cI.x * x00.x - cI.y * g0.x, cI.x * x00.y - cI.y * g0.y);
      cf y10 = make_float2(cI.y * x00.x + cI.x * g0.x, cI.y * x00.y + cI.x * g0.y);
      cf y01 = make_float2(cI.x * x01.x - cI.y * g1.x, cI.x * x01.y - cI.y * g1.y);
      cf y11 = make_float2(cI.y * x01.x + cI.x * g1.x, cI.y * x01.y + cI.x * g1.y);
      x00 = y00; x01 = y01; x10 = y10; x11 = y11;
    }
    if (s00) x00.y = -x00.y;
    if (s01) x01.y = -x01.y;
    if (s10) x10.y = -x10.y;
    if (s11) x11.y = -x11.y;
    A[i00] = x00;
    if (qJok) A[i01] = x01;
    if (qIok) A[i10] = x10;
    if (qIok && qJok) A[i11] = x11;
  };
  int sweep = 0;
  bool converged = (n < 2);
  for (; sweep < P.max_sweeps && !converged; ++sweep) {
    int rotated_this_sweep = 0;
    for (int stage = 0; stage < m - 1; ++stage) {
      // (1) rotation parameters, logged
      bool act = false;
      if (tid < half) {
        int p, q;
        jac_pair(m, stage, tid, p, q);
        JacRot R; R.c = 1.f; R.s = 0.f; R.gx = 1.f; R.gy = 0.f; R.npp = 0.f; R.nqq = 0.f;
        if (q < n) {
          float a = A[(size_t)p * ld + p].x, d = A[(size_t)q * ld + q].x;
          cf b = A[(size_t)p * ld + q];
          float b2 = b.x * b.x + b.y * b.y;
          if (b2 > thr2 && b2 > 0.f) {
            jac_rotation_fast(a, d, b, b2, R);
            act = true;
          }
        }
        rotc[tid] = make_float4(R.c, R.s, R.gx, R.gy);
        rotd[tid] = make_float2(R.npp, R.nqq);
        rotp[tid] = make_int2(act ? p : -1 - p, q);
        md.log[((size_t)sweep * (m - 1) + stage) * half + tid] = make_float4(R.c, R.s, R.gx, R.gy);
      }
      const int applied = __syncthreads_count(act);
      rotated_this_sweep += applied;
      if (applied && worker) {
        // (2) every 2 x 2 block of the upper triangle
        for (int r = I0; r < R; r += rpp) {
          if (r <= cc) do_block(r, cc); else do_block(he - 1 - r, he - 1 - cc);
          if (r == cc) do_block(he - 1 - r, he - 1 - r);
        }
      }
      __syncthreads();
    }
    converged = (rotated_this_sweep == 0);
  }
  if (tid == 0) {
    P.flags[1 + md.index] = sweep;
    if (!converged) atomicOr(&P.flags[0], 1);
  }
  for (int i = tid; i < n; i += nt) md.lam[i] = A[(size_t)i * ld + i].x;
}

// NP = pairs per lane (>= n/64), D = stages of the log kept in flight
template <int NP, int D>
__global__ void __launch_bounds__(256) jacobi_vectors_kernel(JacobiFastParams P) {
  extern __shared__ __align__(16) unsigned char jvs[];
  cf* rows = reinterpret_cast<cf*>(jvs);                    // [8][row_stride]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * 8 + warp;
  if (gw >= P.total_rows) return;
  int mi = 0;
  for (int i = 1; i < P.nmodes; ++i) if (gw >= P.mode[i].row0) mi = i;
  const JacobiFastMode md = P.mode[mi];
  if (P.flags[JAC_SKIP + md.index]) return;
  const int n = md.n, i_row = gw - md.row0;
  const int m = (n + 1) & ~1, half = m >> 1;
  const int sweeps = P.flags[1 + md.index];
  cf* row = rows + (size_t)warp * P.row_stride;
  for (int j = lane; j < n; j += 32) row[j] = make_float2(j == i_row ? 1.f : 0.f, 0.f);
  __syncwarp();
  // the log is replayed D stages at a time, the next D already in flight
  const float4* lg = md.log;
  const int nst = sweeps * (m - 1);
  const float4 ident = make_float4(1.f, 0.f, 1.f, 0.f);
  float4 cur[D][NP], nxt[D][NP];
  auto fetch = [&](float4 (&buf)[D][NP], int s0) {
#pragma unroll
    for (int d = 0; d < D; ++d)
#pragma unroll
      for (int e = 0; e < NP; ++e) {
        const int tb = lane + 32 * e;
        buf[d][e] = (s0 + d < nst && tb < half) ? lg[(size_t)(s0 + d) * half + tb] : ident;
      }
  };
  fetch(cur, 0);
  int stage = 0;
  for (int s0 = 0; s0 < nst; s0 += D) {
    fetch(nxt, s0 + D);
#pragma unroll
    for (int d = 0; d < D; ++d) {
      if (s0 + d < nst) {
#pragma unroll
        for (int e = 0; e < NP; ++e) {
          const float4 R = cur[d][e];
          const int tb = lane + 32 * e;
          if (tb >= half || (R.y == 0.f && R.x == 1.f && R.z == 1.f && R.w == 0.f)) continue;      // identity
          int p, q;
          jac_pair(m, stage, tb, p, q);
          cf xp = row[p], xq = row[q];
          cf gq = make_float2(R.z * xq.x - R.w * xq.y, R.z * xq.y + R.w * xq.x);
          row[p] = make_float2(R.x * xp.x - R.y * gq.x, R.x * xp.y - R.y * gq.y);
          row[q] = make_float2(R.y * xp.x + R.x * gq.x, R.y * xp.y + R.x * gq.y);
        }
        __syncwarp();
        if (++stage == m - 1) stage = 0;
      }
    }
#pragma unroll
    for (int d = 0; d < D; ++d)
#pragma unroll
      for (int e = 0; e < NP; ++e) cur[d][e] = nxt[d][e];
  }
  for (int j = lane; j < n; j += 32) md.V[(size_t)i_row * n + j] = row[j];
}

__global__ void __launch_bounds__(JAC_THREADS) jacobi_factors_kernel(JacobiFastParams P) {
  const JacobiFastMode md = P.mode[blockIdx.x];
  if (P.flags[JAC_SKIP + md.index]) return;
  const int n = md.n, r = md.r;
  const cf* __restrict__ V = md.V;
  __shared__ float lam[JAC_FAST_MAX_N];
  __shared__ int rank_of[JAC_FAST_MAX_N];
  const int tid = threadIdx.x, nt = blockDim.x;
  for (int i = tid; i < n; i += nt) lam[i] = md.lam[i];
  __syncthreads();
  for (int i = tid; i < n; i += nt) {
    float li = lam[i]; int rk = 0;
    for (int j = 0; j < n; ++j) { float lj = lam[j]; rk += (lj > li) || (lj == li && j < i); }
    rank_of[i] = rk;
  }
  __syncthreads();
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
