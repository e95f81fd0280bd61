// Mode-n products on the small intermediate tensors of the Tucker chain, and
// the Adam update of the core.
//
// A tensor is viewed as [O][K][C] (O = product of the modes before n, C =
// product of the modes after n, contiguous).  The mode-n product
//   out[o][m][c] = sum_k Aop[m][k] in[o][k][c]
// (Definition "Mode-k Product") uses Aop = U^H (M = r_n, K = I_n) when
// compressing and Aop = U (M = I_n, K = r_n) when reconstructing; U is the
// I_n x r_n row-major factor matrix in both cases.
#pragma once
#include "common.cuh"
#include "tail.cuh"

namespace tg {

constexpr int MP_BM = 32, MP_BC = 64, MP_BK = 16;

template <bool CONJ_T>
__global__ void __launch_bounds__(256) mode_product_kernel(const cf* __restrict__ in, cf* __restrict__ out,
                                                           const cf* __restrict__ U, int M, int K, int C, int r_n) {
  __shared__ __align__(16) cf As[MP_BK][MP_BM];
  __shared__ __align__(16) cf Bs[MP_BK][MP_BC];
  const int tid = threadIdx.x;
  const int tm = tid >> 4, tc = tid & 15;          // 16 x 16 threads: 2 rows (m) x 4 cols (c) each
  const int m0 = blockIdx.y * MP_BM, c0 = blockIdx.x * MP_BC;
  const size_t o = blockIdx.z;
  const cf* inb = in + o * (size_t)K * C;
  cf acc[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.f, 0.f);

  for (int k0 = 0; k0 < K; k0 += MP_BK) {
    // A tile: As[kk][mm] = Aop[m0+mm][k0+kk]
    for (int i = tid; i < MP_BK * MP_BM; i += 256) {
      int kk, mm;
      if (CONJ_T) { mm = i % MP_BM; kk = i / MP_BM; }   // U[k][m]: m contiguous
      else { kk = i % MP_BK; mm = i / MP_BK; }          // U[m][k]: k contiguous
      int m = m0 + mm, k = k0 + kk;
      cf v = make_float2(0.f, 0.f);
      if (m < M && k < K) {
        if (CONJ_T) { cf u = U[(size_t)k * r_n + m]; v = make_float2(u.x, -u.y); }
        else v = U[(size_t)m * r_n + k];
      }
      As[kk][mm] = v;
    }
    for (int i = tid; i < MP_BK * MP_BC; i += 256) {
      int cc = i % MP_BC, kk = i / MP_BC;
      int c = c0 + cc, k = k0 + kk;
      Bs[kk][cc] = (c < C && k < K) ? inb[(size_t)k * C + c] : make_float2(0.f, 0.f);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < MP_BK; ++kk) {
      cf a[2], b[4];
      load_row_bcast<2>(&As[kk][tm * 2], a);
      load_row_bcast<4>(&Bs[kk][tc * 4], b);
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) cfma(acc[i][j], a[i], b[j]);
    }
    __syncthreads();
  }
  cf* outb = out + o * (size_t)M * C;
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    int m = m0 + tm * 2 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int c = c0 + tc * 4 + j;
      if (c < C) outb[(size_t)m * C + c] = acc[i][j];
    }
  }
}

// AdamUpdate of Algorithm 1 on the Tucker core: moments in place, N_L out.
__global__ void adam_core_kernel(const cf* __restrict__ core, cf* __restrict__ m_l, float* __restrict__ v_l,
                                 cf* __restrict__ n_l, uint32_t n, AdamScalars a) {
  uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    cf m = m_l[i]; float v = v_l[i];
    cf r = adam_apply(core[i], m, v, a);
    m_l[i] = m; v_l[i] = v; n_l[i] = r;
  }
}

}  // namespace tg
