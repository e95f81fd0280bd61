// The two full-tensor streaming kernels of a step.
//
// The tensor is seen as S = prod(I_1..I_{N-2}) slabs of A x B entries
// (A = I_{N-1}, B = I_N, B contiguous).  This file holds what all variants share (parameters, the
// AdamUpdate) and the general kernels: one thread block per slab at a time, fp32 arithmetic, any
// slab that fits in shared memory, any storage type.
//
// proj_tail (read G once):   per slab, gather the sparse values at Omega (their Adam update runs with
//   the core's), zero them (the residual R = G - Sparse(G, Omega)), then
//   contract the two trailing modes:  T[s, ja, jb] = sum_{a,b} conj(Ua[a,ja]) conj(Ub[b,jb]) R[s,a,b]
//   (the last two of the chained mode-n products of the low-rank compression).
// back_tail (read+write W once): per slab, expand the two trailing modes of the
//   normalised core, D[s,a,b] = sum_{ja,jb} Ua[a,ja] Ub[b,jb] T'[s,ja,jb], and apply
//   W <- (1 - eta wd) W - eta alpha D, then W[Omega] -= eta lambda N_S
//   (reconstruction, scaled sparse add and weight update of Algorithm 1).
#pragma once
#include "common.cuh"

namespace tg {

struct AdamScalars {
  float beta1, beta2, omb1, omb2;   // decay rates and (1 - beta)
  float inv_c1, inv_c2;             // 1 / (1 - beta^(t+1))
  float eps;
};

// One Adam update in the compressed space (AdamUpdate of Algorithm 1; |x conj(x)|
// for the second moment).  Returns the normalised update N.
__device__ __forceinline__ cf adam_apply(cf x, cf& m, float& v, const AdamScalars& a) {
  m.x = a.beta1 * m.x + a.omb1 * x.x;
  m.y = a.beta1 * m.y + a.omb1 * x.y;
  v = a.beta2 * v + a.omb2 * (x.x * x.x + x.y * x.y);
  float den = sqrtf(v * a.inv_c2) + a.eps;
  float sc = a.inv_c1 / den;
  return make_float2(m.x * sc, m.y * sc);
}

struct TailParams {
  int A, B, Bs;          // slab rows, cols, padded smem row stride (odd)
  int ra, rb, ras;       // ranks of the two trailing modes; padded smem row stride of Ua (odd)
  uint32_t nslab, E;     // number of slabs, A*B
  const cf* Ua;          // U^(N-1), A x ra row-major
  const cf* Ub;          // U^(N),   B x rb row-major
  const uint32_t* omega; // ascending flat indices
  const uint32_t* slab_ptr; // slab_ptr[s] = first Omega slot of slab s (nslab + 1 entries)
  int k;
  int keep;              // compression: 1 = gather the entries at Omega but leave them in place (the low-rank part sees
                         // the gradient itself, not the residual of the sparse part)
  cf* m_s; float* v_s;   // sparse moments (proj)
  cf* g_s;               // gathered sparse values (fast path: their Adam update runs in the Adam kernel)
  cf* n_s;               // normalised sparse update: written by proj, read by back
  cf* t;                 // proj: out T[s][ra][rb];  back: in T'[s][ra][rb]
  AdamScalars adam;
  float s_low, s_sparse; // eta*alpha, eta*lambda
  float decay;           // 1 - eta*wd
};

template <int RBP>
__device__ __forceinline__ void load_row_bcast(const cf* __restrict__ row, cf (&u)[RBP]) {
  // row is 16-byte aligned and RBP is a multiple of 2
  const float4* p = reinterpret_cast<const float4*>(row);
#pragma unroll
  for (int j = 0; j < RBP / 2; ++j) {
    float4 q = p[j];
    u[2 * j] = make_float2(q.x, q.y);
    u[2 * j + 1] = make_float2(q.z, q.w);
  }
}

// ---------------------------------------------------------------------------------------------
// General streaming kernels (any slab shape that fits in shared memory, both storage types): one
// thread block per slab at a time, fp32 FMA arithmetic.  Shared memory (units of cf):
//   X/W slab [A][Bs] | Y [A][rbp] | Ub [B][rbp] | (back) T' [ra][rbp] | (back) Ua [A][ras]
// Bs, ras odd (conflict-free column walks); rbp = rb rounded up to a multiple of 8.
// ---------------------------------------------------------------------------------------------
constexpr int TB_THREADS = 256;
constexpr int TB_YR = 16;        // Y entries a thread keeps in registers in the last product of the reconstruction

struct TailBlkGeom {
  int Bs, rbp, ras, js;          // padded strides; js = threads per slab row in the products over b
  uint32_t off_y, off_ub, off_t, off_ua, total;   // byte offsets
};
__host__ inline TailBlkGeom tail_blk_geom(int A, int B, int ra, int rb, bool back) {
  TailBlkGeom g;
  g.Bs = B | 1; g.rbp = (rb + 7) & ~7; g.ras = ra | 1; g.js = g.rbp / 8;
  size_t o = (size_t)A * g.Bs * 8; o = (o + 15) & ~(size_t)15;
  g.off_y = (uint32_t)o; o += (size_t)A * g.rbp * 8;
  g.off_ub = (uint32_t)o; o += (size_t)B * g.rbp * 8;
  g.off_t = (uint32_t)o; if (back) o += (size_t)ra * g.rbp * 8;
  g.off_ua = (uint32_t)o; if (back) o += (((size_t)A * g.ras * 8) + 15) & ~(size_t)15;
  g.total = (uint32_t)o;
  return g;
}

// Compression of the two trailing modes of one slab at a time, fused with the sparse gather and the
// residual:  Y[a][jb] = sum_b R[a][b] conj(Ub[b][jb]),  T[ja][jb] = sum_a conj(Ua[a][ja]) Y[a][jb].
// The gathered sparse values go to p.g_s (their AdamUpdate runs with the core's).
template <class S>
__global__ void __launch_bounds__(TB_THREADS) proj_tail_blk_kernel(const void* __restrict__ g, TailParams p, TailBlkGeom G) {
  griddep_chain();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int A = p.A, B = p.B, Bs = G.Bs, ra = p.ra, rb = p.rb, rbp = G.rbp, js = G.js;
  cf* xs = reinterpret_cast<cf*>(smem_raw);
  cf* ys = reinterpret_cast<cf*>(smem_raw + G.off_y);
  cf* ubs = reinterpret_cast<cf*>(smem_raw + G.off_ub);      // conj(Ub), zero padded
  for (int i = tid; i < B * rbp; i += TB_THREADS) {
    const int b = i / rbp, j = i - b * rbp;
    cf u = (j < rb) ? p.Ub[b * rb + j] : make_float2(0.f, 0.f);
    ubs[i] = make_float2(u.x, -u.y);
  }
  const uint32_t E = p.E;
  const int rows_pp = TB_THREADS / js, arow = tid / js, jq = (tid - arow * js) * 8;
  for (uint32_t s = blockIdx.x; s < p.nslab; s += gridDim.x) {
    const size_t gbase = (size_t)s * E;
    __syncthreads();                                     // the previous slab's products are done with xs / ys
    for (int a = warp; a < A; a += TB_THREADS / 32)
      for (int b = lane; b < B; b += 32) xs[a * Bs + b] = S::load(g, gbase + (size_t)a * B + b);
    __syncthreads();
    if (p.k > 0) {
      const int j0 = (int)p.slab_ptr[s], j1 = (int)p.slab_ptr[s + 1];
      for (int j = j0 + tid; j < j1; j += TB_THREADS) {
        const uint32_t loc = p.omega[j] - (uint32_t)gbase;
        const uint32_t a = loc / B;
        const uint32_t si = a * Bs + (loc - a * B);
        p.g_s[j] = xs[si];
        if (!p.keep) xs[si] = make_float2(0.f, 0.f);
      }
      __syncthreads();
    }
    // ---- mode N: a thread owns 8 consecutive jb of one row ----
    for (int a = arow; a < A; a += rows_pp) {
      cf acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = make_float2(0.f, 0.f);
      const cf* xr = xs + a * Bs;
      for (int b = 0; b < B; ++b) {
        const cf x = xr[b];
        cf u[8];
        load_row_bcast<8>(ubs + b * rbp + jq, u);
#pragma unroll
        for (int j = 0; j < 8; ++j) cfma(acc[j], x, u[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) ys[a * rbp + jq + j] = acc[j];
    }
    __syncthreads();
    // ---- mode N-1: one output T[ja][jb] per thread and pass ----
    cf* tout = p.t + (size_t)s * ra * rb;
    for (int o = tid; o < ra * rb; o += TB_THREADS) {
      const int ja = o / rb, jb = o - ja * rb;
      cf acc = make_float2(0.f, 0.f);
#pragma unroll 4
      for (int a = 0; a < A; ++a) cfma_conj(acc, ys[a * rbp + jb], __ldg(&p.Ua[a * ra + ja]));   // y * conj(u)
      tout[o] = acc;
    }
  }
}

// Reconstruction of the two trailing modes of one slab at a time, fused with the weight update and the
// sparse add:  Y'[a][jb] = sum_ja Ua[a][ja] T'[ja][jb],  D[a][b] = sum_jb Y'[a][jb] Ub[b][jb],
// W <- (1 - eta wd) W - eta alpha D, then W[Omega] -= eta lambda N_S (half storage: the dense result is
// rounded to fp16 before the sparse term is added, and once more when stored).
template <class S>
__global__ void __launch_bounds__(TB_THREADS) back_tail_blk_kernel(void* __restrict__ w, TailParams p, TailBlkGeom G) {
  griddep_chain();
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int A = p.A, B = p.B, Bs = G.Bs, ra = p.ra, rb = p.rb, rbp = G.rbp, ras = G.ras, js = G.js;
  cf* ws = reinterpret_cast<cf*>(smem_raw);
  cf* ys = reinterpret_cast<cf*>(smem_raw + G.off_y);
  cf* ubs = reinterpret_cast<cf*>(smem_raw + G.off_ub);      // Ub, zero padded
  cf* ts = reinterpret_cast<cf*>(smem_raw + G.off_t);
  cf* uas = reinterpret_cast<cf*>(smem_raw + G.off_ua);
  for (int i = tid; i < B * rbp; i += TB_THREADS) {
    const int b = i / rbp, j = i - b * rbp;
    ubs[i] = (j < rb) ? p.Ub[b * rb + j] : make_float2(0.f, 0.f);
  }
  for (int i = tid; i < A * ra; i += TB_THREADS) {
    const int a = i / ra, j = i - a * ra;
    uas[a * ras + j] = p.Ua[i];
  }
  const uint32_t E = p.E;
  const bool decay = p.decay != 1.0f;
  const int rows_pp = TB_THREADS / js, arow = tid / js, jq = (tid - arow * js) * 8;
  // last product: tpr threads share a row, each walks every tpr-th column
  const int tpr = (A >= TB_THREADS) ? 1 : TB_THREADS / A, rows_pp2 = TB_THREADS / tpr;
  const int arow2 = tid / tpr, bq = tid - arow2 * tpr;
  for (uint32_t s = blockIdx.x; s < p.nslab; s += gridDim.x) {
    const size_t gbase = (size_t)s * E;
    __syncthreads();                                     // the previous slab has been stored
    for (int a = warp; a < A; a += TB_THREADS / 32)
      for (int b = lane; b < B; b += 32) {
        cf v = S::load(w, gbase + (size_t)a * B + b);
        if (decay) { v.x *= p.decay; v.y *= p.decay; }
        ws[a * Bs + b] = v;
      }
    {
      const cf* tin = p.t + (size_t)s * ra * rb;
      for (int i = tid; i < ra * rbp; i += TB_THREADS) {
        const int ja = i / rbp, j = i - ja * rbp;
        ts[i] = (j < rb) ? tin[ja * rb + j] : make_float2(0.f, 0.f);
      }
    }
    __syncthreads();
    // ---- mode N-1: a thread owns 8 consecutive jb of one row ----
    for (int a = arow; a < A; a += rows_pp) {
      cf acc[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[j] = make_float2(0.f, 0.f);
      const cf* ur = uas + a * ras;
      for (int ja = 0; ja < ra; ++ja) {
        const cf u = ur[ja];
        cf tv[8];
        load_row_bcast<8>(ts + ja * rbp + jq, tv);
#pragma unroll
        for (int j = 0; j < 8; ++j) cfma(acc[j], u, tv[j]);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) ys[a * rbp + jq + j] = acc[j];
    }
    __syncthreads();
    // ---- mode N: Y'[a][.] in registers (TB_YR at a time), applied to the row column by column ----
    for (int a = arow2; a < A; a += rows_pp2) {
      for (int jc = 0; jc < rbp; jc += TB_YR) {
        cf y[TB_YR];
#pragma unroll
        for (int j = 0; j < TB_YR; j += 8) {
          if (jc + j < rbp) load_row_bcast<8>(ys + a * rbp + jc + j, *reinterpret_cast<cf(*)[8]>(&y[j]));
          else {
#pragma unroll
            for (int q = 0; q < 8; ++q) y[j + q] = make_float2(0.f, 0.f);
          }
        }
        for (int b = bq; b < B; b += tpr) {
          cf d = make_float2(0.f, 0.f);
#pragma unroll
          for (int j = 0; j < TB_YR; j += 8) {
            if (jc + j < rbp) {
              cf u[8];
              load_row_bcast<8>(ubs + b * rbp + jc + j, u);
#pragma unroll
              for (int q = 0; q < 8; ++q) cfma(d, y[j + q], u[q]);
            }
          }
          cf wv = ws[a * Bs + b];
          wv.x = fmaf(-p.s_low, d.x, wv.x); wv.y = fmaf(-p.s_low, d.y, wv.y);
          ws[a * Bs + b] = wv;
        }
      }
    }
    __syncthreads();
    // ---- scaled sparse add at Omega (on top of the dense update) ----
    if (p.k > 0) {
      const int j0 = (int)p.slab_ptr[s], j1 = (int)p.slab_ptr[s + 1];
      for (int j = j0 + tid; j < j1; j += TB_THREADS) {
        const uint32_t loc = p.omega[j] - (uint32_t)gbase;
        const uint32_t a = loc / B;
        const uint32_t si = a * Bs + (loc - a * B);
        cf wv = ws[si];
        wv = S::narrow(wv);
        const cf n = p.n_s[j];
        wv.x = fmaf(-p.s_sparse, n.x, wv.x); wv.y = fmaf(-p.s_sparse, n.y, wv.y);
        ws[si] = wv;
      }
      __syncthreads();
    }
    for (int a = warp; a < A; a += TB_THREADS / 32)
      for (int b = lane; b < B; b += 32) S::store(w, gbase + (size_t)a * B + b, ws[a * Bs + b]);
  }
}

}  // namespace tg
