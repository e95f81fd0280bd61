// Leading eigenvectors of the Gram matrices A_n by subspace iteration with Rayleigh-Ritz steps.
//
// TuckerFactors of Algorithm 1 needs, per mode, only the eigenvectors of the r_n largest eigenvalues of
// A_n = R_(n) R_(n)^H (I_n x I_n, Hermitian PSD), and between two refreshes that subspace usually moves
// little (the appendix "Tensor Decomposition / Implementation" restarts the decomposition from the previous
// factors for that reason).  A full Jacobi diagonalisation of A_n does I_n / r_n times more work than that
// and runs on one SM per mode.  Here, per mode and in one thread block:
//
//   Q <- orthonormal n x R start, R = r + a few guard columns: the previous U^(n) (warm) or a fixed
//        pseudo-random matrix (cold), completed by pseudo-random columns
//   repeat:  Z <- A Q,  H <- Q^H Z
//            a Rayleigh-Ritz step when it is due (see below): eigen-decomposition of the small H by cyclic
//            Jacobi in shared memory, Q <- Q W with the columns in eigenvalue order (Ritz vectors), Z <- A Q,
//            residuals rho_j = || Z_j - theta_j Q_j ||;  stop when
//            max_{j<r} rho_j <= SUB_TOL (theta_r - theta_{r+1})
//            (the sine of the largest angle to the invariant subspace is at most rho / gap)
//            Z <- T_d(L) Q, the Chebyshev polynomial of odd degree d <= 7 of L = (2/b) A - I, which maps the
//            unwanted part [0, b] of the spectrum into [-1, 1] and grows like cosh(d acosh(x)) above it
//            (b: the largest Rayleigh quotient among the guard columns; d: the smallest degree whose growth at
//            the r-th eigenvalue covers the reduction still needed; d = 1 is the plain power step);  a
//            spectrum whose wanted and unwanted parts are close, lambda_{r+1} / lambda_r = 0.8 say, converges
//            at 0.42 per multiplication this way instead of 0.8
//            Q <- orthonormalisation of Z (Cholesky of the column-scaled Z^H Z; Gram-Schmidt if that breaks down)
//   The small Jacobi is the expensive part (one SM, two barriers per rotation stage), so a Rayleigh-Ritz step is
//   only taken (i) once after three multiplications of a cold start, to sort the basis, and (ii) when the
//   residual of the leading r columns against their own span, || Z_r - Q_r H_rr ||, is below the target --
//   the orthonormalisation keeps the column order, so those columns keep spanning the leading subspace.
//   All matrix products run on the tensor cores (split-precision TF32, fp32 accumulation).
//
// The result is the same eigen-decomposition the Jacobi path computes (same order, same canonical phase), to
// the stated angle.  Whenever the iteration cannot certify that -- no gap after r eigenvalues, a (numerically)
// rank-deficient or non-finite matrix, the small Jacobi hitting its sweep cap, the iteration cap -- it leaves
// the mode's "done" word at 0 and the full Jacobi kernels, which are always launched after it and return at
// once for the modes that are done, take over.  Every loop is bounded.
#pragma once
#include "common.cuh"
#include "jacobi.cuh"
#include "ptx.cuh"

namespace tg {

constexpr int SUB_THREADS = 1024;
constexpr int SUB_MAX_N = 256;            // rows of Q that fit beside the small matrices in shared memory
constexpr int SUB_MAX_R = 80;
constexpr int SUB_MAX_IT = 12;            // outer iterations (each up to SUB_MAX_DEG multiplications by A) before giving up
// Unsigned key that orders like the float, with every NaN below -inf.
__device__ __forceinline__ uint32_t sub_order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
constexpr int SUB_MAX_DEG = 7;            // highest degree of the polynomial filter
constexpr float SUB_MAX_GROWTH = 1e6f;    // cap on the filter's amplification of the largest eigenvalue (fp32 range of a column)
constexpr float SUB_TOL = 1e-4f;          // bound on the sine of the largest angle to the invariant subspace
constexpr int SUB_DONE = 16;              // flags[SUB_DONE + mode]: 1 = this refresh's U^(n) is already written

struct SubspaceMode {
  const cf* A;        // n x n, row-major (both triangles stored)
  cf* U;              // in (warm start: the previous factor) / out: n x r
  cf* Zg;             // n x ldz scratch in global memory, used when Z does not fit in shared memory
  int n, r, R;
  int index;          // tensor mode
  int z_in_smem;
};
struct SubspaceParams {
  SubspaceMode mode[8];
  int nmodes;
  int warm;           // start from the factors stored in U
  int max_sweeps;     // cap of the small Jacobi
  float tol;          // its off-diagonal tolerance relative to the largest diagonal entry
  int* flags;         // flags[1 + mode]: iterations used; flags[SUB_DONE + mode]
};

// guard columns beside the r wanted ones: they make the convergence rate lambda_{R+1} / lambda_r instead of
// lambda_{r+1} / lambda_r and give the Ritz value that estimates lambda_{r+1} in the stopping test
__host__ __device__ inline int sub_guard(int r) { return (r <= 16 || r >= 48) ? 4 : 8; }
__host__ __device__ inline int sub_ld(int R) { return R | 1; }         // odd row length: column walks spread over the banks
__host__ __device__ inline size_t sub_smem(int n, int R, bool z_in_smem) {
  const size_t ld = (size_t)sub_ld(R);
  const size_t half = (size_t)((R + 1) / 2);
  size_t b = (size_t)n * ld * sizeof(cf) * (z_in_smem ? 2 : 1);        // Q (and Z)
  b += 2 * (size_t)R * ld * sizeof(cf);                                 // H, W
  b += (size_t)n * sizeof(cf) + (size_t)R * (sizeof(cf) + sizeof(float) + sizeof(int));   // v, c, theta, order
  b += half * (sizeof(float4) + sizeof(float2) + sizeof(int2)) + 64 * sizeof(float) + 16;
  b += (size_t)(SUB_THREADS / 32) * R * sizeof(float);                 // per-warp partial residual sums
  return (b + 15) & ~(size_t)15;
}
// whether the mode is handled here at all: guard columns must exist and everything must fit
__host__ __device__ inline bool sub_eligible(int n, int r, int& R, bool& z_in_smem) {
  R = r + sub_guard(r);
  if (R >= n || n > SUB_MAX_N || R > SUB_MAX_R) return false;
  z_in_smem = sub_smem(n, R, true) <= (size_t)200 * 1024;
  return sub_smem(n, R, z_in_smem) <= (size_t)226 * 1024;
}

// fixed pseudo-random value in [-1, 1) from an integer hash of (mode, row, column, part)
__device__ __forceinline__ float sub_rand(uint32_t a, uint32_t b, uint32_t c, uint32_t part) {
  uint32_t h = a * 0x9E3779B1u ^ (b + 0x7F4A7C15u) * 0x85EBCA77u ^ (c + 0x165667B1u) * 0xC2B2AE3Du ^ part * 0x27D4EB2Fu;
  h ^= h >> 15; h *= 0x2C1B3C6Du; h ^= h >> 12; h *= 0x297A2D39u; h ^= h >> 15;
  return (float)(int32_t)h * (1.0f / 2147483648.0f);
}

// barrier over the first n threads of the block (n a multiple of 32), and the same with a count of true predicates
__device__ __forceinline__ void sub_bar(int n) { asm volatile("barrier.sync 1, %0;" ::"r"(n) : "memory"); }
__device__ __forceinline__ int sub_bar_count(int n, bool pred) {
  int r;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %2, 0;\n\t"
      "barrier.red.popc.u32 %0, 1, %1, p;\n\t}"
      : "=r"(r)
      : "r"(n), "r"((int)pred)
      : "memory");
  return r;
}
constexpr int SUB_JT = 512;               // threads that run the small Jacobi (measured: 128 and 256 slower, 1024 the same)

__device__ __forceinline__ void sub_split(float x, float& hi, float& lo) {
  hi = __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
  lo = x - hi;
}

// One warp: tot[q] = op(A)[rows 8 mt .. 8 mt + 7][0..K) * B[0..K)[columns 8 (nt0 + q) .. + 7], q < NG, complex, as
// split-precision TF32 MMAs (rows g <-> (m, re), g + 8 <-> (m, im); k = t <-> (k, re), t + 4 <-> (k, im); n = g <-> c).
// AT = false: op(A)[m][k] = A[m lda + k];  AT = true: op(A)[m][k] = conj(A[k lda + m]).  B is row-major, K x N.
// Out of range rows, columns and k read as zero.  Result: tot[q][0] + i tot[q][2] = C[8 mt + g][8 (nt0 + q) + 2 t],
// tot[q][1] + i tot[q][3] = the entry to its right.
template <bool AT, int NG>
__device__ __forceinline__ void sub_tile_product(const cf* A, int lda, const cf* B, int ldb, int M, int N, int K,
                                                 int mt, int nt0, int lane, float (&tot)[NG][4]) {
  const int g = lane >> 2, t = lane & 3;
  float d[NG][4];
#pragma unroll
  for (int q = 0; q < NG; ++q)
#pragma unroll
    for (int e = 0; e < 4; ++e) { tot[q][e] = 0.f; d[q][e] = 0.f; }
  const int m = 8 * mt + g;
  auto load_a = [&](int k) -> cf {
    cf a = make_float2(0.f, 0.f);
    if (m < M && k < K) {
      if (AT) { const cf u = A[(size_t)k * lda + m]; a = make_float2(u.x, -u.y); }
      else a = A[(size_t)m * lda + k];
    }
    return a;
  };
  // 16 k at a time: the four A fragments are requested together (A may live in global memory), and the MMA
  // accumulators, whose adds truncate, are emptied into round-to-nearest sums after each such group
  for (int k0 = 0; k0 < K; k0 += 16) {
    cf av[4];
#pragma unroll
    for (int s_ = 0; s_ < 4; ++s_) av[s_] = load_a(k0 + 4 * s_ + t);
#pragma unroll
    for (int s_ = 0; s_ < 4; ++s_) {
      const int k = k0 + 4 * s_ + t;
      float arh, arl, aih, ail;
      sub_split(av[s_].x, arh, arl); sub_split(av[s_].y, aih, ail);
#pragma unroll
      for (int q = 0; q < NG; ++q) {
        const int c = 8 * (nt0 + q) + g;
        const cf x = (k < K && c < N) ? B[(size_t)k * ldb + c] : make_float2(0.f, 0.f);
        float xh0, xl0, xh1, xl1;
        sub_split(x.x, xh0, xl0); sub_split(x.y, xh1, xl1);
        mma_tf32(d[q], arh, aih, -aih, arh, xh0, xh1);
        mma_tf32(d[q], arl, ail, -ail, arl, xh0, xh1);
        mma_tf32(d[q], arh, aih, -aih, arh, xl0, xl1);
      }
    }
#pragma unroll
    for (int q = 0; q < NG; ++q)
#pragma unroll
      for (int e = 0; e < 4; ++e) { tot[q][e] += d[q][e]; d[q][e] = 0.f; }
  }
#pragma unroll
  for (int q = 0; q < NG; ++q)
#pragma unroll
    for (int e = 0; e < 4; ++e) tot[q][e] += d[q][e];
}

// The whole block: C = op(A) B, every 8 x 8 tile handed to `out(row, col, c0, c1)` (the entries at (row, col) and
// (row, col + 1); the callee checks the range).  A warp takes one tile row and NG tile columns at a time.
template <bool AT, class F>
__device__ __forceinline__ void sub_gemm(const cf* A, int lda, const cf* B, int ldb, int M, int N, int K, int warp,
                                         int lane, int nwarps, F out) {
  constexpr int NG = 3;
  const int mtiles = (M + 7) >> 3, ntiles = (N + 7) >> 3, ngroups = (ntiles + NG - 1) / NG;
  const int g = lane >> 2, t = lane & 3;
  for (int task = warp; task < mtiles * ngroups; task += nwarps) {
    const int mt = task / ngroups, nt0 = (task - mt * ngroups) * NG;
    float tot[NG][4];
    sub_tile_product<AT, NG>(A, lda, B, ldb, M, N, K, mt, nt0, lane, tot);
#pragma unroll
    for (int q = 0; q < NG; ++q)
      out(8 * mt + g, 8 * (nt0 + q) + 2 * t, make_float2(tot[q][0], tot[q][2]), make_float2(tot[q][1], tot[q][3]));
  }
}

__global__ void __launch_bounds__(SUB_THREADS, 1) subspace_kernel(SubspaceParams P) {
  extern __shared__ __align__(16) unsigned char ssm[];
  const SubspaceMode md = P.mode[blockIdx.x];
  const int n = md.n, r = md.r, R = md.R, ld = sub_ld(R);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NW = SUB_THREADS / 32;
  const int m = (R + 1) & ~1, half = m >> 1;
  // ---- shared memory ----
  cf* Q = reinterpret_cast<cf*>(ssm);                                   // [n][ld]
  cf* Zs = Q + (size_t)n * ld;
  cf* Hm = Zs + (md.z_in_smem ? (size_t)n * ld : 0);                    // [R][ld]
  cf* Wm = Hm + (size_t)R * ld;                                         // [R][ld]
  cf* vcol = Wm + (size_t)R * ld;                                       // [n]
  cf* ccoef = vcol + n;                                                 // [R]
  float* theta = reinterpret_cast<float*>(ccoef + R);                   // [R]
  int* order = reinterpret_cast<int*>(theta + R);                       // [R]: order[j] = index of the j-th largest
  float4* rotc = reinterpret_cast<float4*>((reinterpret_cast<uintptr_t>(order + R) + 15) & ~(uintptr_t)15);
  float2* rotd = reinterpret_cast<float2*>(rotc + half);
  int2* rotp = reinterpret_cast<int2*>(rotd + half);
  float* red = reinterpret_cast<float*>(rotp + half);                   // [64]
  float* respart = red + 64;                                            // [NW][R]
  cf* Z = md.z_in_smem ? Zs : md.Zg;                                    // generic pointer: shared or global
  const int ldz = ld;

  // block-wide sum of one float per thread; the result is returned to every thread
  auto block_sum = [&](float x) -> float {
    for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();
    if (lane == 0) red[warp] = x;
    __syncthreads();
    float s = 0.f;
    for (int w = 0; w < NW; ++w) s += red[w];
    return s;
  };

  // rows are spread over lane groups: `parts` threads share a row
  int npad = 32; while (npad < n) npad <<= 1;
  const int parts = SUB_THREADS / npad;                                 // power of two, 4 .. 32
  const int urow = tid / parts, upart = tid - urow * parts;

  // ---- Q <- orthonormalised Z by classical Gram-Schmidt applied twice, column by column (slow: one column at a
  //      time with block barriers, but indifferent to the conditioning of Z); false if a column has nothing new ----
  auto orthonormalise_gs = [&]() -> bool {
    for (int j = 0; j < R; ++j) {
      for (int i = tid; i < n; i += SUB_THREADS) vcol[i] = Z[(size_t)i * ldz + j];
      __syncthreads();
      float n0 = 0.f;
      for (int i = tid; i < n; i += SUB_THREADS) { const cf v = vcol[i]; n0 += v.x * v.x + v.y * v.y; }
      n0 = block_sum(n0);
      for (int pass = 0; pass < 2 && j > 0; ++pass) {
        for (int jj = warp; jj < j; jj += NW) {                         // c[jj] = Q[:, jj]^H v
          cf acc = make_float2(0.f, 0.f);
          for (int i = lane; i < n; i += 32) cfma_conj(acc, vcol[i], Q[(size_t)i * ld + jj]);
          for (int o = 16; o; o >>= 1) { acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o); }
          if (lane == 0) ccoef[jj] = acc;
        }
        __syncthreads();
        {                                                               // v -= Q[:, :j] c
          cf acc = make_float2(0.f, 0.f);
          if (urow < n)
            for (int jj = upart; jj < j; jj += parts) cfma(acc, Q[(size_t)urow * ld + jj], ccoef[jj]);
          for (int o = parts >> 1; o; o >>= 1) { acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o); }
          if (urow < n && upart == 0) { cf v = vcol[urow]; v.x -= acc.x; v.y -= acc.y; vcol[urow] = v; }
        }
        __syncthreads();
      }
      float n1 = 0.f;
      for (int i = tid; i < n; i += SUB_THREADS) { const cf v = vcol[i]; n1 += v.x * v.x + v.y * v.y; }
      n1 = block_sum(n1);
      if (!(n1 > 1e-10f * n0) || !(n1 > 1e-37f) || !(n1 < 3e38f)) return false;      // also catches NaN
      const float inv = rsqrtf(n1);
      for (int i = tid; i < n; i += SUB_THREADS) { const cf v = vcol[i]; Q[(size_t)i * ld + j] = make_float2(v.x * inv, v.y * inv); }
      __syncthreads();
    }
    return true;
  };

  // ---- the same by Cholesky: G = X^H X = L L^H, Q = X L^-H (X = Z in the first pass, Q itself in the second, which
  //      removes what the first leaves when X is not well conditioned).  false if a pivot shows that G is too
  //      ill-conditioned for this to work in fp32 (the caller then takes the Gram-Schmidt route). ----
  auto cholesky_pass = [&](const cf* X, int ldx) -> bool {
    sub_gemm<true>(X, ldx, X, ldx, R, R, n, warp, lane, NW, [&](int a, int b, cf c0, cf c1) {
      if (a < R && b < R) Hm[(size_t)a * ld + b] = c0;
      if (a < R && b + 1 < R) Hm[(size_t)a * ld + b + 1] = c1;
    });
    __syncthreads();
    // scale to unit diagonal (the columns of a filtered block differ by orders of magnitude): G <- D G D, D = diag(G)^-1/2
    for (int j = tid; j < R; j += SUB_THREADS) { const float gjj = Hm[(size_t)j * ld + j].x; theta[j] = gjj > 0.f ? rsqrtf(gjj) : 0.f; }
    __syncthreads();
    for (int idx = tid; idx < R * R; idx += SUB_THREADS) {
      const int a = idx / R, b = idx - a * R;
      const float sc = theta[a] * theta[b];
      cf v = Hm[(size_t)a * ld + b]; v.x *= sc; v.y *= sc;
      Hm[(size_t)a * ld + b] = v;
    }
    __syncthreads();
    if (warp == 0) {
      // left-looking, one warp: column j of L from column j of G and the columns before it
      bool good = true;
      for (int j = 0; j < R; ++j) {
        for (int i = j + lane; i < R; i += 32) {
          cf acc = Hm[(size_t)i * ld + j];
          if (i == j) acc.y = 0.f;
          for (int k2 = 0; k2 < j; ++k2) {
            const cf a = Hm[(size_t)i * ld + k2], b = Hm[(size_t)j * ld + k2];
            acc.x -= a.x * b.x + a.y * b.y; acc.y -= a.y * b.x - a.x * b.y;          // acc -= L[i][k] conj(L[j][k])
          }
          Hm[(size_t)i * ld + j] = acc;
        }
        __syncwarp();
        const float pivot = Hm[(size_t)j * ld + j].x;
        float g0 = 0.f;                                                 // the diagonal entry as it was: pivot + |L[j][:j]|^2
        for (int k2 = lane; k2 < j; k2 += 32) { const cf b = Hm[(size_t)j * ld + k2]; g0 += b.x * b.x + b.y * b.y; }
        for (int o = 16; o; o >>= 1) g0 += __shfl_xor_sync(0xffffffffu, g0, o);
        g0 += pivot;
        if (!(pivot > 1e-5f * g0) || !(pivot < 3e38f)) { good = false; break; }       // uniform in the warp
        const float ljj = sqrtf(pivot), inv = 1.f / ljj;
        for (int i = j + 1 + lane; i < R; i += 32) { const cf v = Hm[(size_t)i * ld + j]; Hm[(size_t)i * ld + j] = make_float2(v.x * inv, v.y * inv); }
        if (lane == 0) Hm[(size_t)j * ld + j] = make_float2(ljj, 0.f);
        __syncwarp();
      }
      if (lane == 0) red[63] = good ? 1.f : 0.f;
    }
    __syncthreads();
    if (red[63] == 0.f) return false;
    // q[j] = (x[j] - sum_{k<j} q[k] conj(L[j][k])) / L[j][j], row by row; `parts` lanes share a row
    for (int j = 0; j < R; ++j) {
      cf acc = make_float2(0.f, 0.f);
      if (urow < n)
        for (int k2 = upart; k2 < j; k2 += parts) cfma_conj(acc, Q[(size_t)urow * ld + k2], Hm[(size_t)j * ld + k2]);
      for (int o = parts >> 1; o; o >>= 1) { acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o); }
      if (urow < n && upart == 0) {
        cf x = X[(size_t)urow * ldx + j];
        x.x *= theta[j]; x.y *= theta[j];
        const float inv = 1.f / Hm[(size_t)j * ld + j].x;
        Q[(size_t)urow * ld + j] = make_float2((x.x - acc.x) * inv, (x.y - acc.y) * inv);
      }
      __syncwarp();
    }
    __syncthreads();
    return true;
  };
  // One Cholesky pass leaves an orthonormality defect of about cond(Z)^2 2^-24, which the power iteration does not
  // mind; `twice` polishes it away (needed before a Rayleigh-Ritz step, whose Ritz vectors become U^(n)).
  auto orthonormalise = [&](bool twice) -> bool {
    if (cholesky_pass(Z, ldz) && (!twice || cholesky_pass(Q, ld))) return true;
    return orthonormalise_gs();
  };

  auto fill_start = [&](bool warm) {
    for (int idx = tid; idx < n * R; idx += SUB_THREADS) {
      const int i = idx / R, j = idx - i * R;
      cf v;
      if (warm && j < r) v = md.U[(size_t)i * r + j];
      else v = make_float2(sub_rand(md.index, i, j, 0), sub_rand(md.index, i, j, 1));
      Z[(size_t)i * ldz + j] = v;
    }
    __syncthreads();
  };
  auto multiply = [&]() {                                               // Z = A Q
    sub_gemm<false>(md.A, n, Q, ld, n, R, n, warp, lane, NW, [&](int i, int j, cf c0, cf c1) {
      if (i < n && j < R) Z[(size_t)i * ldz + j] = c0;
      if (i < n && j + 1 < R) Z[(size_t)i * ldz + j + 1] = c1;
    });
    __syncthreads();
  };

  // prev <- (4/b) A cur - 2 cur - prev: one step of the Chebyshev recurrence Y_{k+1} = 2 L Y_k - Y_{k-1}
  auto cheb_step = [&](bool into_q, float b) {
    const cf* cur = into_q ? Z : Q;
    const int ldc = into_q ? ldz : ld;
    cf* prev = into_q ? Q : Z;
    const int ldp = into_q ? ld : ldz;
    const float s4 = 4.f / b;
    sub_gemm<false>(md.A, n, cur, ldc, n, R, n, warp, lane, NW, [&](int i, int j, cf c0, cf c1) {
      if (i < n && j < R) {
        const cf y = cur[(size_t)i * ldc + j], o = prev[(size_t)i * ldp + j];
        prev[(size_t)i * ldp + j] = make_float2(s4 * c0.x - 2.f * y.x - o.x, s4 * c0.y - 2.f * y.y - o.y);
      }
      if (i < n && j + 1 < R) {
        const cf y = cur[(size_t)i * ldc + j + 1], o = prev[(size_t)i * ldp + j + 1];
        prev[(size_t)i * ldp + j + 1] = make_float2(s4 * c1.x - 2.f * y.x - o.x, s4 * c1.y - 2.f * y.y - o.y);
      }
    });
    __syncthreads();
  };
  // T_d(x) for odd d, x >= 1
  auto cheb_growth = [](int d, float x) -> float {
    const float x2 = x * x;
    if (d <= 1) return x;
    if (d == 3) return x * (4.f * x2 - 3.f);
    if (d == 5) return x * ((16.f * x2 - 20.f) * x2 + 5.f);
    return x * (((64.f * x2 - 112.f) * x2 + 56.f) * x2 - 7.f);
  };

  float tr_a = 0.f;
  for (int i = tid; i < n; i += SUB_THREADS) tr_a += md.A[(size_t)i * n + i].x;
  tr_a = block_sum(tr_a);

  bool ok;
  fill_start(P.warm != 0);
  ok = orthonormalise(true);
  bool sorted = P.warm != 0;     // the leading r columns are (about) the leading subspace: true for a stored factor
  if (!ok && P.warm) { fill_start(false); ok = orthonormalise(true); sorted = false; }      // unusable stored factor: start cold
  bool polished = true;          // Q is orthonormal to rounding (two passes)

  bool done = false;
  int it = 0;
  while (ok && !done && it < SUB_MAX_IT) {
    ++it;
    multiply();
    // ---- H = Q^H Z, made exactly Hermitian ----
    auto rayleigh = [&]() {
      sub_gemm<true>(Q, ld, Z, ldz, R, R, n, warp, lane, NW, [&](int a, int b, cf c0, cf c1) {
        if (a < R && b < R) Hm[(size_t)a * ld + b] = c0;
        if (a < R && b + 1 < R) Hm[(size_t)a * ld + b + 1] = c1;
      });
      __syncthreads();
      for (int idx = tid; idx < R * R; idx += SUB_THREADS) {
        const int a = idx / R, b = idx - a * R;
        if (a > b) continue;
        const cf u = Hm[(size_t)a * ld + b], l = Hm[(size_t)b * ld + a];
        const cf h = make_float2(0.5f * (u.x + l.x), a == b ? 0.f : 0.5f * (u.y - l.y));
        Hm[(size_t)a * ld + b] = h;
        Hm[(size_t)b * ld + a] = make_float2(h.x, -h.y);
      }
      __syncthreads();
    };
    rayleigh();
    bool ritz = (it == SUB_MAX_IT);                                     // the last chance
    // what the filter needs: b = upper end of the unwanted spectrum, lam_w = the smallest wanted eigenvalue (estimates),
    // lam_1 = the largest, need = the factor by which the wanted part still has to outgrow the rest
    float cheb_b = 0.f, lam_w = 0.f, lam_1 = 0.f, need = 3e38f;
    {
      float tr_h = 0.f, dm = 0.f;
      for (int j = 0; j < R; ++j) { const float dj = Hm[(size_t)j * ld + j].x; tr_h += dj; dm = fmaxf(dm, dj); }
      lam_1 = dm;
      if (!sorted) { cheb_b = (tr_a - tr_h) / (float)(n - R); lam_w = cheb_b; }     // mean eigenvalue outside span(Q); all of Q is wanted
    }
    if (!sorted) ritz = ritz || (it == 2);
    else {
      // ---- residual of the leading r columns against their own span: E = Z_r - Q_r H_rr, column norms ----
      for (int idx = tid; idx < NW * R; idx += SUB_THREADS) respart[idx] = 0.f;
      __syncthreads();
      sub_gemm<false>(Q, ld, Hm, ld, n, r, r, warp, lane, NW, [&](int i, int j, cf c0, cf c1) {
        float e0 = 0.f, e1 = 0.f;
        if (i < n && j < r) { const cf z = Z[(size_t)i * ldz + j]; const float dx = z.x - c0.x, dy = z.y - c0.y; e0 = dx * dx + dy * dy; }
        if (i < n && j + 1 < r) { const cf z = Z[(size_t)i * ldz + j + 1]; const float dx = z.x - c1.x, dy = z.y - c1.y; e1 = dx * dx + dy * dy; }
        // sum over the tile's eight rows (lanes that differ in g), then one lane per column pair adds
        for (int o = 4; o < 32; o <<= 1) { e0 += __shfl_xor_sync(0xffffffffu, e0, o); e1 += __shfl_xor_sync(0xffffffffu, e1, o); }
        if ((lane >> 2) == 0) {
          if (j < r) respart[warp * R + j] += e0;
          if (j + 1 < r) respart[warp * R + j + 1] += e1;
        }
        __syncwarp();
      });
      __syncthreads();
      float worst = 0.f, dlo = 3e38f, dhi = 0.f;
      for (int j = tid; j < R; j += SUB_THREADS) {
        const float dj = Hm[(size_t)j * ld + j].x;
        if (j < r) {
          float sres = 0.f;
          for (int w = 0; w < NW; ++w) sres += respart[w * R + j];
          worst = fmaxf(worst, sres);
          dlo = fminf(dlo, dj);
        } else dhi = fmaxf(dhi, dj);
      }
      for (int o = 16; o; o >>= 1) {
        worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, o));
        dlo = fminf(dlo, __shfl_xor_sync(0xffffffffu, dlo, o));
        dhi = fmaxf(dhi, __shfl_xor_sync(0xffffffffu, dhi, o));
      }
      if (lane == 0) { red[warp] = worst; red[32 + warp] = (warp < (R + 31) / 32) ? dlo : 3e38f; }
      __syncthreads();
      worst = 0.f; dlo = 3e38f;
      for (int w = 0; w < NW; ++w) { worst = fmaxf(worst, red[w]); dlo = fminf(dlo, red[32 + w]); }
      __syncthreads();
      if (lane == 0) red[warp] = dhi;
      __syncthreads();
      dhi = 0.f;
      for (int w = 0; w < NW; ++w) dhi = fmaxf(dhi, red[w]);
      const float gap = dlo - dhi;                                      // diagonal entries stand in for Ritz values here
      ritz = ritz || (gap > 0.f && worst <= (0.5f * SUB_TOL * gap) * (0.5f * SUB_TOL * gap));
      cheb_b = dhi; lam_w = dlo;
      need = gap > 0.f ? 4.f * sqrtf(worst) / (SUB_TOL * gap) : 3e38f;
      __syncthreads();
    }
    if (ritz) {
      if (!polished) {
        // the Ritz vectors inherit the orthonormality of Q: second Cholesky pass now, then Z and H again
        if (!cholesky_pass(Q, ld)) { ok = false; break; }
        polished = true;
        multiply();
        rayleigh();
      }
      // ---- cyclic Jacobi on H (R x R, full storage), rotations accumulated in W; run by the first SUB_JT
      //      threads, the others wait at the block barrier below ----
      for (int idx = tid; idx < R * R; idx += SUB_THREADS) {
        const int a = idx / R, b = idx - a * R;
        Wm[(size_t)a * ld + b] = make_float2(a == b ? 1.f : 0.f, 0.f);
      }
      __syncthreads();
      if (tid < SUB_JT) {
        float dmax = 0.f;
        for (int i = tid; i < R; i += SUB_JT) dmax = fmaxf(dmax, fabsf(Hm[(size_t)i * ld + i].x));
        for (int o = 16; o; o >>= 1) dmax = fmaxf(dmax, __shfl_xor_sync(0xffffffffu, dmax, o));
        if (lane == 0) red[32 + warp] = dmax;
        sub_bar(SUB_JT);
        dmax = 0.f;
        for (int w = 0; w < SUB_JT / 32; ++w) dmax = fmaxf(dmax, red[32 + w]);
        const float thr2 = (P.tol * dmax) * (P.tol * dmax);
        bool conv = false;
        for (int sweep = 0; sweep < P.max_sweeps && !conv; ++sweep) {
          int rotated = 0;
          for (int stage = 0; stage < m - 1; ++stage) {
            bool act = false;
            if (tid < half) {
              int p, q;
              jac_pair(m, stage, tid, p, q);
              JacRot Rt; Rt.c = 1.f; Rt.s = 0.f; Rt.gx = 1.f; Rt.gy = 0.f; Rt.npp = 0.f; Rt.nqq = 0.f;
              if (q < R) {
                const float a = Hm[(size_t)p * ld + p].x, d = Hm[(size_t)q * ld + q].x;
                const cf b = Hm[(size_t)p * ld + q];
                const float b2 = b.x * b.x + b.y * b.y;
                if (b2 > thr2 && b2 > 0.f) { jac_rotation_fast(a, d, b, b2, Rt); act = true; }
              }
              rotc[tid] = make_float4(Rt.c, Rt.s, Rt.gx, Rt.gy);
              rotd[tid] = make_float2(Rt.npp, Rt.nqq);
              rotp[tid] = make_int2(act ? p : -1 - p, q);
            }
            const int applied = sub_bar_count(SUB_JT, act);
            rotated += applied;
            if (applied) {
              // every 2 x 2 block (I, J) of H: columns by the rotation of pair J, rows by that of pair I
              for (int task = tid; task < half * half; task += SUB_JT) {
                const int I = task / half, J = task - I * half;
                const int2 pqI = rotp[I], pqJ = rotp[J];
                if (pqI.x < 0 && pqJ.x < 0) continue;
                const int pI = pqI.x < 0 ? -1 - pqI.x : pqI.x, qI = pqI.y, pJ = pqJ.x < 0 ? -1 - pqJ.x : pqJ.x, qJ = pqJ.y;
                if (I == J) {
                  const float2 dd = rotd[I];
                  Hm[(size_t)pI * ld + pI] = make_float2(dd.x, 0.f);
                  Hm[(size_t)qI * ld + qI] = make_float2(dd.y, 0.f);
                  Hm[(size_t)pI * ld + qI] = make_float2(0.f, 0.f);
                  Hm[(size_t)qI * ld + pI] = make_float2(0.f, 0.f);
                  continue;
                }
                const float4 cI = rotc[I], cJ = rotc[J];
                const bool qIok = qI < R, qJok = qJ < R;
                const cf z = make_float2(0.f, 0.f);
                cf x00 = Hm[(size_t)pI * ld + pJ], x01 = qJok ? Hm[(size_t)pI * ld + qJ] : z;
                cf x10 = qIok ? Hm[(size_t)qI * ld + pJ] : z, x11 = (qIok && qJok) ? Hm[(size_t)qI * ld + qJ] : z;
                {
                  const cf g0 = make_float2(cJ.z * x01.x - cJ.w * x01.y, cJ.z * x01.y + cJ.w * x01.x);
                  const cf g1 = make_float2(cJ.z * x11.x - cJ.w * x11.y, cJ.z * x11.y + cJ.w * x11.x);
                  const cf y00 = make_float2(cJ.x * x00.x - cJ.y * g0.x, cJ.x * x00.y - cJ.y * g0.y);
                  const cf y01 = make_float2(cJ.y * x00.x + cJ.x * g0.x, cJ.y * x00.y + cJ.x * g0.y);
                  const cf y10 = make_float2(cJ.x * x10.x - cJ.y * g1.x, cJ.x * x10.y - cJ.y * g1.y);
                  const cf y11 = make_float2(cJ.y * x10.x + cJ.x * g1.x, cJ.y * x10.y + cJ.x * g1.y);
                  x00 = y00; x01 = y01; x10 = y10; x11 = y11;
                }
                {
                  const cf g0 = make_float2(cI.z * x10.x + cI.w * x10.y, cI.z * x10.y - cI.w * x10.x);
                  const cf g1 = make_float2(cI.z * x11.x + cI.w * x11.y, cI.z * x11.y - cI.w * x11.x);
                  const cf y00 = make_float2(cI.x * x00.x - cI.y * g0.x, cI.x * x00.y - cI.y * g0.y);
                  const cf y10 = make_float2(cI.y * x00.x + cI.x * g0.x, cI.y * x00.y + cI.x * g0.y);
                  const cf y01 = make_float2(cI.x * x01.x - cI.y * g1.x, cI.x * x01.y - cI.y * g1.y);
                  const cf y11 = make_float2(cI.y * x01.x + cI.x * g1.x, cI.y * x01.y + cI.x * g1.y);
                  x00 = y00; x01 = y01; x10 = y10; x11 = y11;
                }
                Hm[(size_t)pI * ld + pJ] = x00;
                if (qJok) Hm[(size_t)pI * ld + qJ] = x01;
                if (qIok) Hm[(size_t)qI * ld + pJ] = x10;
                if (qIok && qJok) Hm[(size_t)qI * ld + qJ] = x11;
              }
              // W <- W J: columns (p, q) of every row
              for (int task = tid; task < R * half; task += SUB_JT) {
                const int i = task / half, J = task - i * half;
                const int2 pq = rotp[J];
                if (pq.x < 0 || pq.y >= R) continue;
                const float4 c = rotc[J];
                const cf xp = Wm[(size_t)i * ld + pq.x], xq = Wm[(size_t)i * ld + pq.y];
                const cf gq = make_float2(c.z * xq.x - c.w * xq.y, c.z * xq.y + c.w * xq.x);
                Wm[(size_t)i * ld + pq.x] = make_float2(c.x * xp.x - c.y * gq.x, c.x * xp.y - c.y * gq.y);
                Wm[(size_t)i * ld + pq.y] = make_float2(c.y * xp.x + c.x * gq.x, c.y * xp.y + c.x * gq.y);
              }
            }
            sub_bar(SUB_JT);
          }
          conv = (rotated == 0);
        }
        if (tid == 0) red[62] = conv ? 1.f : 0.f;
      }
      __syncthreads();
      if (red[62] == 0.f) { ok = false; break; }
      // ---- Ritz values in descending order (ties: lower index first) ----
      for (int i = tid; i < R; i += SUB_THREADS) theta[i] = Hm[(size_t)i * ld + i].x;
      __syncthreads();
      // (compared through sub_order_key: a strict total order even with NaN among the values, so that the ranks
      // are a permutation and every order[] entry is written)
      for (int i = tid; i < R; i += SUB_THREADS) {
        const uint32_t li = sub_order_key(theta[i]);
        int rk = 0;
        for (int j = 0; j < R; ++j) { const uint32_t lj = sub_order_key(theta[j]); rk += (lj > li) || (lj == li && j < i); }
        order[rk] = i;
      }
      __syncthreads();
      // ---- Q <- Q W with the columns in that order (through the Z buffer), then Z <- A Q again ----
      for (int idx = tid; idx < R * R; idx += SUB_THREADS) {
        const int a = idx / R, b = idx - a * R;
        Hm[(size_t)a * ld + b] = Wm[(size_t)a * ld + order[b]];
      }
      __syncthreads();
      sub_gemm<false>(Q, ld, Hm, ld, n, R, R, warp, lane, NW, [&](int i, int j, cf c0, cf c1) {
        if (i < n && j < R) Z[(size_t)i * ldz + j] = c0;
        if (i < n && j + 1 < R) Z[(size_t)i * ldz + j + 1] = c1;
      });
      __syncthreads();
      for (int idx = tid; idx < n * R; idx += SUB_THREADS) {
        const int i = idx / R, j = idx - i * R;
        Q[(size_t)i * ld + j] = Z[(size_t)i * ldz + j];
      }
      __syncthreads();
      multiply();
      sorted = true;
      // ---- residuals rho_j^2 = || Z_j - theta_j Q_j ||^2 of the r leading Ritz pairs ----
      for (int j = warp; j < r; j += NW) {
        const float th = theta[order[j]];
        float sres = 0.f;
        for (int i = lane; i < n; i += 32) {
          const cf z = Z[(size_t)i * ldz + j], q = Q[(size_t)i * ld + j];
          const float dx = z.x - th * q.x, dy = z.y - th * q.y;
          sres += dx * dx + dy * dy;
        }
        for (int o = 16; o; o >>= 1) sres += __shfl_xor_sync(0xffffffffu, sres, o);
        if (lane == 0) respart[j] = sres;
      }
      __syncthreads();
      float worst = 0.f;
      for (int j = 0; j < r; ++j) worst = fmaxf(worst, respart[j]);
      const float gap = theta[order[r - 1]] - theta[order[r]];
      done = gap > 0.f && worst <= (SUB_TOL * gap) * (SUB_TOL * gap);      // false for NaN
      cheb_b = theta[order[r]]; lam_w = theta[order[r - 1]]; lam_1 = theta[order[0]];
      need = gap > 0.f ? 4.f * sqrtf(worst) / (SUB_TOL * gap) : 3e38f;
      __syncthreads();
      if (done) break;
    }
    // ---- the filter: Z = T_d((2/b) A - I) Q, starting from Z = A Q ----
    if (cheb_b > 0.f && cheb_b < 3e38f && lam_w > cheb_b * 1.0001f) {
      const float xw = (2.f * lam_w - cheb_b) / cheb_b, x1 = fmaxf(xw, (2.f * lam_1 - cheb_b) / cheb_b);
      int d = 1;
      while (d < SUB_MAX_DEG && cheb_growth(d, xw) < need) d += 2;
      while (d > 1 && cheb_growth(d, x1) > SUB_MAX_GROWTH) d -= 2;
      if (d > 1) {
        const float s2 = 2.f / cheb_b;
        for (int idx = tid; idx < n * R; idx += SUB_THREADS) {
          const int i = idx / R, j = idx - i * R;
          const cf z = Z[(size_t)i * ldz + j], q = Q[(size_t)i * ld + j];
          Z[(size_t)i * ldz + j] = make_float2(s2 * z.x - q.x, s2 * z.y - q.y);       // Y_1 = L Q
        }
        __syncthreads();
        for (int k = 1; k < d; ++k) cheb_step((k & 1) != 0, cheb_b);       // Y_2 lands in Q, Y_3 in Z, ...: odd d ends in Z
      }
    }
    ok = orthonormalise(false);
    polished = false;
  }
  if (tid == 0) P.flags[SUB_DONE + md.index] = done ? 1 : 0;
  if (!done) return;
  if (tid == 0) P.flags[1 + md.index] = it;
  // ---- U = the first r Ritz vectors, each scaled by the unit phase that makes its largest-modulus component
  //      real positive (first such row on ties) ----
  for (int j = warp; j < r; j += NW) {
    float best = -1.f; int bi = 0;
    for (int a = lane; a < n; a += 32) {
      const cf v = Q[(size_t)a * ld + j];
      const float mg = v.x * v.x + v.y * v.y;
      if (mg > best) { best = mg; bi = a; }
    }
    for (int o = 16; o; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    const cf pv = Q[(size_t)bi * ld + j];
    const float mg = sqrtf(pv.x * pv.x + pv.y * pv.y);
    const cf ph = mg > 0.f ? make_float2(pv.x / mg, -pv.y / mg) : make_float2(1.f, 0.f);
    for (int a = lane; a < n; a += 32) {
      const cf v = Q[(size_t)a * ld + j];
      md.U[(size_t)a * r + j] = make_float2(v.x * ph.x - v.y * ph.y, v.x * ph.y + v.y * ph.x);
    }
  }
}

}  // namespace tg
