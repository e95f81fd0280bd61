// Mode-n products on the small intermediate tensors of the Tucker chain, and
// the Adam update of the core.
//
// A tensor is viewed as [O][K][C] (O = product of the modes before n, C =
// product of the modes after n, contiguous).  The mode-n product
//   out[o][m][c] = sum_k Aop[m][k] in[o][k][c]
// (Definition "Mode-k Product") uses Aop = U^H (M = r_n, K = I_n) when
// compressing and Aop = U (M = I_n, K = r_n) when reconstructing; U is the
// I_n x r_n row-major factor matrix in both cases.
//
// These tensors are at most a few tens of MB and stay in L2, so the kernel is
// bound by fp32 FMA issue: a block of 128 threads owns a 32 (m) x 64 (c) output
// tile, a thread a 4 x 4 complex micro-tile (64 real FMAs per k for 4 shared
// loads of 16 bytes); the next k-slice is fetched into registers while the
// current one is being multiplied.
#pragma once
#include "common.cuh"
#include "tail.cuh"

namespace tg {

constexpr int MP_BM = 32, MP_BC = 64, MP_BK = 16, MP_THREADS = 128;

template <bool CONJ_T>
__global__ void __launch_bounds__(MP_THREADS) mode_product_kernel(const cf* __restrict__ in, cf* __restrict__ out,
                                                                  const cf* __restrict__ U, int M, int K, int C, int r_n) {
  __shared__ __align__(16) cf As[2][MP_BK][MP_BM];
  __shared__ __align__(16) cf Bs[2][MP_BK][MP_BC];
  const int tid = threadIdx.x;
  const int tm = tid >> 4, tc = tid & 15;          // 8 x 16 threads: 4 rows (m) x 4 cols (c) each
  const int m0 = blockIdx.y * MP_BM, c0 = blockIdx.x * MP_BC;
  const size_t o = blockIdx.z;
  const cf* inb = in + o * (size_t)K * C;
  constexpr int A_PER = MP_BK * MP_BM / MP_THREADS;   // 4
  constexpr int B_PER = MP_BK * MP_BC / MP_THREADS;   // 8
  cf ra[A_PER], rb[B_PER];

  auto fetch = [&](int k0) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int idx = tid + i * MP_THREADS;
      int kk, mm;
      if (CONJ_T) { mm = idx % MP_BM; kk = idx / MP_BM; }   // U[k][m]: m contiguous
      else { kk = idx % MP_BK; mm = idx / MP_BK; }          // U[m][k]: k contiguous
      const int m = m0 + mm, k = k0 + kk;
      cf v = make_float2(0.f, 0.f);
      if (m < M && k < K) {
        if (CONJ_T) { cf u = U[(size_t)k * r_n + m]; v = make_float2(u.x, -u.y); }
        else v = U[(size_t)m * r_n + k];
      }
      ra[i] = v;
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int idx = tid + i * MP_THREADS;
      const int cc = idx % MP_BC, kk = idx / MP_BC;
      const int c = c0 + cc, k = k0 + kk;
      rb[i] = (c < C && k < K) ? inb[(size_t)k * C + c] : make_float2(0.f, 0.f);
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int i = 0; i < A_PER; ++i) {
      const int idx = tid + i * MP_THREADS;
      int kk, mm;
      if (CONJ_T) { mm = idx % MP_BM; kk = idx / MP_BM; }
      else { kk = idx % MP_BK; mm = idx / MP_BK; }
      As[buf][kk][mm] = ra[i];
    }
#pragma unroll
    for (int i = 0; i < B_PER; ++i) {
      const int idx = tid + i * MP_THREADS;
      Bs[buf][idx / MP_BC][idx % MP_BC] = rb[i];
    }
  };

  cf acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.f, 0.f);

  fetch(0);
  stash(0);
  __syncthreads();
  int buf = 0;
  for (int k0 = 0; k0 < K; k0 += MP_BK) {
    const bool more = k0 + MP_BK < K;
    if (more) fetch(k0 + MP_BK);
#pragma unroll
    for (int kk = 0; kk < MP_BK; ++kk) {
      cf a[4], b[4];
      load_row_bcast<4>(&As[buf][kk][tm * 4], a);
      load_row_bcast<4>(&Bs[buf][kk][tc * 4], b);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) cfma(acc[i][j], a[i], b[j]);
    }
    if (more) stash(buf ^ 1);
    __syncthreads();
    buf ^= 1;
  }
  cf* outb = out + o * (size_t)M * C;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + tm * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = c0 + tc * 4 + j;
      if (c < C) outb[(size_t)m * C + c] = acc[i][j];
    }
  }
}

// AdamUpdate of Algorithm 1 on the Tucker core (entries [0, n)) and, when the streaming kernel only
// gathered them, on the ks sparse values (entries [n, n + ks)): moments in place, N_L / N_S out.
__global__ void adam_kernel(const cf* __restrict__ core, cf* __restrict__ m_l, float* __restrict__ v_l,
                            cf* __restrict__ n_l, uint32_t n, const cf* __restrict__ g_s, cf* __restrict__ m_s,
                            float* __restrict__ v_s, cf* __restrict__ n_s, uint32_t ks, AdamScalars a) {
  uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    cf m = m_l[i]; float v = v_l[i];
    cf r = adam_apply(core[i], m, v, a);
    m_l[i] = m; v_l[i] = v; n_l[i] = r;
  } else if (i - n < ks) {
    i -= n;
    cf m = m_s[i]; float v = v_s[i];
    cf r = adam_apply(g_s[i], m, v, a);
    m_s[i] = m; v_s[i] = v; n_s[i] = r;
  }
}

}  // namespace tg
