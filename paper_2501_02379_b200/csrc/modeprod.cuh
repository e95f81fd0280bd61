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
// These tensors are at most a few tens of MB and stay in L2.  The products run on
// the tensor cores as split-precision TF32 (mode_product_tc_kernel); products with
// very few output rows and small slices use an fp32 kernel that keeps a whole slice
// in shared memory (mode_product_small_kernel); the first mode is fused with the
// AdamUpdate of the core (core_sandwich_tc_kernel).
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "tail.cuh"

namespace tg {

// ---------------------------------------------------------------------------------------------
// The product for few output rows (M <= 8) and slices whose K C entries fit in shared memory: the 32-row
// tensor-core tiles would be mostly padding there.  A block walks over slices o;
// the slice [K][C] and Aop sit in shared memory, a thread owns outputs (m, c) and sums over k in fp32.
// ---------------------------------------------------------------------------------------------
constexpr int MS_THREADS = 256;
__host__ __device__ inline size_t mode_small_smem(int M, int K, int C) { return ((size_t)K * C + (size_t)M * K) * sizeof(cf); }

template <bool CONJ_T>
__global__ void __launch_bounds__(MS_THREADS) mode_product_small_kernel(const cf* __restrict__ in, cf* __restrict__ out,
                                                                        const cf* __restrict__ U, int M, int K, int C,
                                                                        int r_n, int O) {
  extern __shared__ __align__(16) unsigned char msm[];
  cf* Xs = reinterpret_cast<cf*>(msm);           // [K][C]
  cf* As = Xs + (size_t)K * C;                   // [M][K]
  const int tid = threadIdx.x;
  for (int idx = tid; idx < M * K; idx += MS_THREADS) {
    const int m = idx / K, k = idx - m * K;
    cf v;
    if (CONJ_T) { const cf u = U[(size_t)k * r_n + m]; v = make_float2(u.x, -u.y); }
    else v = U[(size_t)m * r_n + k];
    As[idx] = v;
  }
  griddep_chain();            // the factor alone was read so far
  const int KC = K * C, MC = M * C;
  for (int o = blockIdx.x; o < O; o += gridDim.x) {
    const cf* xin = in + (size_t)o * KC;
    for (int idx = tid; idx < KC; idx += MS_THREADS) Xs[idx] = xin[idx];
    __syncthreads();
    cf* xout = out + (size_t)o * MC;
    for (int idx = tid; idx < MC; idx += MS_THREADS) {
      const int m = idx / C, c = idx - m * C;
      const cf* a = As + (size_t)m * K;
      cf acc = make_float2(0.f, 0.f);
#pragma unroll 4
      for (int k = 0; k < K; ++k) cfma(acc, a[k], Xs[k * C + c]);
      xout[idx] = acc;
    }
    __syncthreads();
  }
}

// AdamUpdate of Algorithm 1 on the Tucker core (entries [0, n)) and, when the streaming kernel only
// gathered them, on the ks sparse values (entries [n, n + ks)): moments in place, N_L / N_S out.
__global__ void adam_kernel(const cf* __restrict__ core, cf* __restrict__ m_l, float* __restrict__ v_l,
                            cf* __restrict__ n_l, uint32_t n, const cf* __restrict__ g_s, cf* __restrict__ m_s,
                            float* __restrict__ v_s, cf* __restrict__ n_s, uint32_t ks, AdamScalars a) {
  griddep_chain();
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

// ---------------------------------------------------------------------------------------------
// The product on the tensor cores, split-precision TF32 (hi*hi + lo*hi + hi*lo, fp32
// accumulation).  Real formulation with the rows of the output doubled instead of its columns:
//   [out_re; out_im][m][c] = [[Ar, -Ai], [Ai, Ar]][m][k] . [Xr; Xi][k][c]
// so that one 8-byte load of the complex entry X[k][c] is a whole B fragment (k = t <-> (k, re),
// k = t+4 <-> (k, im), n = g <-> c) and one complex entry of Aop a whole A fragment
// (rows g <-> (m, re), g+8 <-> (m, im)).  One MMA = 8 m x 8 c x 4 k complex.
// A block of 4 warps owns 32 (m) x 32 NT (c); a warp 32 x 8 NT.  X tiles arrive by 8-byte
// asynchronous copies, double buffered; the Aop tile is stored already split.
// ---------------------------------------------------------------------------------------------
constexpr int MT_BM = 32, MT_BK = 16, MT_THREADS = 128;
constexpr int MT_LDA = 20;                       // float4 per row of the A tile: conflict-free fragment loads

__device__ __forceinline__ void mt_split(float x, float& hi, float& lo) {
  hi = __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
  lo = x - hi;
}

template <bool CONJ_T, int NT>
__global__ void __launch_bounds__(MT_THREADS) mode_product_tc_kernel(const cf* __restrict__ in, cf* __restrict__ out,
                                                                     const cf* __restrict__ U, int M, int K, int C, int r_n) {
  constexpr int BC = 32 * NT, LDX = BC + 4;      // X tile row length: rows 4 slots apart in the 16 bank pairs
  __shared__ __align__(16) float4 As[2][MT_BM][MT_LDA];   // (re.hi, im.hi, re.lo, im.lo) of Aop[m][k]
  __shared__ __align__(16) cf Xs[2][MT_BK][LDX];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  const int m0 = blockIdx.y * MT_BM, c0 = blockIdx.x * BC;
  const size_t o = blockIdx.z;
  const cf* inb = in + o * (size_t)K * C;
  const unsigned char* inbytes = reinterpret_cast<const unsigned char*>(inb);

  cf ra[MT_BK * MT_BM / MT_THREADS];
  auto fetch_a = [&](int k0) {
#pragma unroll
    for (int i = 0; i < MT_BK * MT_BM / MT_THREADS; ++i) {
      const int idx = tid + i * MT_THREADS;
      int kk, mm;
      if (CONJ_T) { mm = idx % MT_BM; kk = idx / MT_BM; } else { kk = idx % MT_BK; mm = idx / MT_BK; }
      const int m = m0 + mm, k = k0 + kk;
      cf v = make_float2(0.f, 0.f);
      if (m < M && k < K) {
        if (CONJ_T) { cf u = U[(size_t)k * r_n + m]; v = make_float2(u.x, -u.y); }
        else v = U[(size_t)m * r_n + k];
      }
      ra[i] = v;
    }
  };
  auto stash_a = [&](int buf) {
#pragma unroll
    for (int i = 0; i < MT_BK * MT_BM / MT_THREADS; ++i) {
      const int idx = tid + i * MT_THREADS;
      int kk, mm;
      if (CONJ_T) { mm = idx % MT_BM; kk = idx / MT_BM; } else { kk = idx % MT_BK; mm = idx / MT_BK; }
      float4 q;
      mt_split(ra[i].x, q.x, q.z); mt_split(ra[i].y, q.y, q.w);
      As[buf][mm][kk] = q;
    }
  };
  auto load_x = [&](int k0, int buf) {
#pragma unroll
    for (int i = 0; i < MT_BK * BC / MT_THREADS; ++i) {
      const int idx = tid + i * MT_THREADS;
      const int cc = idx % BC, kk = idx / BC;
      const int c = c0 + cc, k = k0 + kk;
      const bool v = c < C && k < K;
      cp_async8(&Xs[buf][kk][cc], v ? inbytes + ((size_t)k * C + c) * 8 : inbytes, v ? 8u : 0u);
    }
    cp_async_commit();
  };

  // a warp covers all 4 m-tiles (32 rows = 4 x 8 complex m) and NT column tiles: accumulators [4][NT][4]
  float d[4][NT][4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) d[mt][nt][i] = 0.f;
  // running sums with round-to-nearest adds; the MMA accumulators (whose adds truncate) are emptied into
  // them after every k-slice of 16, i.e. after at most 12 accumulations
  float tot[4][NT][4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) tot[mt][nt][i] = 0.f;

  fetch_a(0);                 // U only: in flight while the previous kernel drains
  griddep_chain();
  load_x(0, 0);
  stash_a(0);
  int buf = 0;
  for (int k0 = 0; k0 < K; k0 += MT_BK, buf ^= 1) {
    cp_async_wait<0>();
    __syncthreads();                               // stage buf is complete; everyone is done with stage buf^1
    const bool more = k0 + MT_BK < K;
    if (more) { fetch_a(k0 + MT_BK); load_x(k0 + MT_BK, buf ^ 1); }
#pragma unroll
    for (int ks = 0; ks < MT_BK / 4; ++ks) {
      const int kc = ks * 4 + t;
      float xh[NT][2], xl[NT][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const cf x = Xs[buf][kc][warp * 8 * NT + nt * 8 + gq];
        mt_split(x.x, xh[nt][0], xl[nt][0]); mt_split(x.y, xh[nt][1], xl[nt][1]);
      }
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) {
        const float4 a = As[buf][mt * 8 + gq][kc];
        // rows (m, re): (Ar | -Ai); rows (m, im): (Ai | Ar)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          mma_tf32(d[mt][nt], a.x, a.y, -a.y, a.x, xh[nt][0], xh[nt][1]);
          mma_tf32(d[mt][nt], a.z, a.w, -a.w, a.z, xh[nt][0], xh[nt][1]);
          mma_tf32(d[mt][nt], a.x, a.y, -a.y, a.x, xl[nt][0], xl[nt][1]);
        }
      }
    }
    if (more) stash_a(buf ^ 1);
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { tot[mt][nt][i] += d[mt][nt][i]; d[mt][nt][i] = 0.f; }
  }
  // d0 = re(m, c = 2t), d1 = re(m, 2t+1), d2 = im(m, 2t), d3 = im(m, 2t+1)
  cf* outb = out + o * (size_t)M * C;
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
    const int m = m0 + mt * 8 + gq;
    if (m >= M) continue;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int c = c0 + warp * 8 * NT + nt * 8 + 2 * t;
      if (c < C) outb[(size_t)m * C + c] = make_float2(tot[mt][nt][0], tot[mt][nt][2]);
      if (c + 1 < C) outb[(size_t)m * C + c + 1] = make_float2(tot[mt][nt][1], tot[mt][nt][3]);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The innermost link of the chain in one launch: last compression product, AdamUpdate of the
// core, first reconstruction product (all three act on columns c of [.][C] independently):
//   core[j][c] = sum_i conj(U1[i][j]) X[i][c]        (mode-1 product with U^(1)H, I_1 -> r_1)
//   N = AdamUpdate(core)                             (moments in place; core and N_L are kept)
//   out[i][c] = sum_j U1[i][j] N[j][c]               (mode-1 product with U^(1), r_1 -> I_1)
// A block takes 16 columns: X[:, block] is read into shared memory before anything is written, so
// `out` may alias `X`.  Blocks past the last column block run the AdamUpdate of the sparse values.
// ---------------------------------------------------------------------------------------------
constexpr int SW_CB = 16, SW_THREADS = 256, SW_MAX_I = 256, SW_MAX_R = 64;
// ---------------------------------------------------------------------------------------------
// Both products run on the tensor cores (split TF32, fragment conventions of mode_product_tc_kernel): the
// whole X[:, 16 columns] block and U1 sit in shared memory, so each product runs without intermediate barriers.
// ---------------------------------------------------------------------------------------------
constexpr int SWT_LDX = SW_CB + 4;      // row length of the X / core tiles: fragment loads hit distinct banks
__host__ __device__ inline int swt_ldu(int r1) { return ((r1 + 7) & ~7) + 4; }
__host__ __device__ inline size_t sandwich_tc_smem(int I1, int r1) {
  const size_t I1p = (size_t)((I1 + 7) & ~7), r1p = (size_t)((r1 + 7) & ~7);
  return (I1p * SWT_LDX + I1p * swt_ldu(r1) + r1p * SWT_LDX) * sizeof(cf);
}

__global__ void __launch_bounds__(SW_THREADS) core_sandwich_tc_kernel(const cf* __restrict__ X, cf* __restrict__ out,
                                                                      const cf* __restrict__ U1, cf* __restrict__ core,
                                                                      cf* __restrict__ m_l, float* __restrict__ v_l,
                                                                      cf* __restrict__ n_l, int I1, int r1, int C,
                                                                      const cf* __restrict__ g_s, cf* __restrict__ m_s,
                                                                      float* __restrict__ v_s, cf* __restrict__ n_s, uint32_t ks,
                                                                      uint32_t nblk_core, AdamScalars a) {
  extern __shared__ __align__(16) unsigned char swm[];
  if (blockIdx.x >= nblk_core) {
    griddep_chain();
    const uint32_t i = (blockIdx.x - nblk_core) * SW_THREADS + threadIdx.x;
    if (i < ks) {
      cf m = m_s[i]; float v = v_s[i];
      cf r = adam_apply(g_s[i], m, v, a);
      m_s[i] = m; v_s[i] = v; n_s[i] = r;
    }
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  const int I1p = (I1 + 7) & ~7, r1p = (r1 + 7) & ~7, ldu = swt_ldu(r1);
  cf* Xs = reinterpret_cast<cf*>(swm);                 // [I1p][SWT_LDX]
  cf* Us = Xs + (size_t)I1p * SWT_LDX;                 // [I1p][ldu], zero padded
  cf* Cs = Us + (size_t)I1p * ldu;                     // [r1p][SWT_LDX]: the core block, then N
  const int c0 = blockIdx.x * SW_CB;
  for (int idx = tid; idx < I1p * (ldu - 4); idx += SW_THREADS) {
    const int i = idx / (ldu - 4), j = idx - i * (ldu - 4);
    Us[i * ldu + j] = (i < I1 && j < r1) ? U1[(size_t)i * r1 + j] : make_float2(0.f, 0.f);
  }
  griddep_chain();            // U1 alone was read so far; X is the previous kernel's output
  {
    // the X block by asynchronous copies (zero-filled outside the tensor); meanwhile this thread's moments
    const unsigned char* xb = reinterpret_cast<const unsigned char*>(X);
    if ((C & 1) == 0) {
      for (int idx = tid; idx < I1p * (SW_CB / 2); idx += SW_THREADS) {
        const int i = idx / (SW_CB / 2), cc = 2 * (idx - i * (SW_CB / 2));
        const bool ok = i < I1 && c0 + cc < C;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(&Xs[i * SWT_LDX + cc])),
                     "l"(ok ? xb + ((size_t)i * C + c0 + cc) * 8 : xb), "r"(ok ? 16u : 0u) : "memory");
      }
    } else {
      for (int idx = tid; idx < I1p * SW_CB; idx += SW_THREADS) {
        const int i = idx / SW_CB, cc = idx - i * SW_CB;
        const bool ok = i < I1 && c0 + cc < C;
        cp_async8(&Xs[i * SWT_LDX + cc], ok ? xb + ((size_t)i * C + c0 + cc) * 8 : xb, ok ? 8u : 0u);
      }
    }
    cp_async_commit();
  }
  // moments of the entries this thread updates after the first product (SW_MAX_R * SW_CB / SW_THREADS = 4 at most)
  constexpr int SW_EPT = SW_MAX_R * SW_CB / SW_THREADS;
  cf pm[SW_EPT]; float pv[SW_EPT];
#pragma unroll
  for (int q = 0; q < SW_EPT; ++q) {
    const int e = tid + q * SW_THREADS, j = e / SW_CB, cc = e - j * SW_CB;
    pm[q] = make_float2(0.f, 0.f); pv[q] = 0.f;
    if (j < r1 && c0 + cc < C) { const size_t idx = (size_t)j * C + c0 + cc; pm[q] = m_l[idx]; pv[q] = v_l[idx]; }
  }
  cp_async_wait<0>();
  __syncthreads();
  // ---- core[j][c] = sum_i conj(U1[i][j]) X[i][c]: rows (j, re|im), k = (i, re|im) ----
  for (int tile = warp; tile < (r1p / 8) * 2; tile += SW_THREADS / 32) {
    const int mt = tile >> 1, nt = tile & 1;
    float tot[4] = {0.f, 0.f, 0.f, 0.f}, acc[4] = {0.f, 0.f, 0.f, 0.f}, acl[4] = {0.f, 0.f, 0.f, 0.f}, acx[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int q = 0; q < I1p / 4; ++q) {
      const int i = 4 * q + t;
      const cf u = Us[i * ldu + 8 * mt + gq], x = Xs[i * SWT_LDX + 8 * nt + gq];
      float urh, url, uih, uil, xh0, xl0, xh1, xl1;
      mt_split(u.x, urh, url); mt_split(u.y, uih, uil);
      mt_split(x.x, xh0, xl0); mt_split(x.y, xh1, xl1);
      // Aop = conj(u): (Ar, Ai) = (ur, -ui); fragment (Ar, Ai, -Ai, Ar); the three products keep their own chains
      mma_tf32(acc, urh, -uih, uih, urh, xh0, xh1);
      mma_tf32(acl, url, -uil, uil, url, xh0, xh1);
      mma_tf32(acx, urh, -uih, uih, urh, xl0, xl1);
      if ((q & 15) == 15) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { tot[e] += acc[e] + (acl[e] + acx[e]); acc[e] = 0.f; acl[e] = 0.f; acx[e] = 0.f; }
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) tot[e] += acc[e] + (acl[e] + acx[e]);
    Cs[(8 * mt + gq) * SWT_LDX + 8 * nt + 2 * t] = make_float2(tot[0], tot[2]);
    Cs[(8 * mt + gq) * SWT_LDX + 8 * nt + 2 * t + 1] = make_float2(tot[1], tot[3]);
  }
  __syncthreads();
  // ---- AdamUpdate of the block (rows past r1 are zero and stay zero) ----
#pragma unroll
  for (int q = 0; q < SW_EPT; ++q) {
    const int e = tid + q * SW_THREADS, j = e / SW_CB, cc = e - j * SW_CB;
    if (j >= r1) break;
    cf n = make_float2(0.f, 0.f);
    if (c0 + cc < C) {
      const size_t idx = (size_t)j * C + c0 + cc;
      const cf x = Cs[j * SWT_LDX + cc];
      cf m = pm[q]; float v = pv[q];
      n = adam_apply(x, m, v, a);
      m_l[idx] = m; v_l[idx] = v; n_l[idx] = n; core[idx] = x;
    }
    Cs[j * SWT_LDX + cc] = n;
  }
  __syncthreads();
  // ---- out[i][c] = sum_j U1[i][j] N[j][c] ----
  for (int tile = warp; tile < (I1p / 8) * 2; tile += SW_THREADS / 32) {
    const int mt = tile >> 1, nt = tile & 1;
    float acc[4] = {0.f, 0.f, 0.f, 0.f}, acl[4] = {0.f, 0.f, 0.f, 0.f}, acx[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
    for (int q = 0; q < r1p / 4; ++q) {
      const int j = 4 * q + t;
      const cf u = Us[(8 * mt + gq) * ldu + j], x = Cs[j * SWT_LDX + 8 * nt + gq];
      float urh, url, uih, uil, xh0, xl0, xh1, xl1;
      mt_split(u.x, urh, url); mt_split(u.y, uih, uil);
      mt_split(x.x, xh0, xl0); mt_split(x.y, xh1, xl1);
      mma_tf32(acc, urh, uih, -uih, urh, xh0, xh1);
      mma_tf32(acl, url, uil, -uil, url, xh0, xh1);
      mma_tf32(acx, urh, uih, -uih, urh, xl0, xl1);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] += acl[e] + acx[e];
    const int i = 8 * mt + gq, c = c0 + 8 * nt + 2 * t;
    if (i < I1) {
      if (c < C) out[(size_t)i * C + c] = make_float2(acc[0], acc[2]);
      if (c + 1 < C) out[(size_t)i * C + c + 1] = make_float2(acc[1], acc[3]);
    }
  }
}

}  // namespace tg
