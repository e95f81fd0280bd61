// The two full-tensor streaming kernels of a step.
//
// The tensor is seen as S = prod(I_1..I_{N-2}) slabs of A x B entries
// (A = I_{N-1}, B = I_N, B contiguous).  One warp owns one slab at a time.
//
// proj_tail (read G once):   per slab, gather the sparse values at Omega and run
//   their Adam update, zero them (the residual R = G - Sparse(G, Omega)), then
//   contract the two trailing modes:  T[s, ja, jb] = sum_{a,b} conj(Ua[a,ja]) conj(Ub[b,jb]) R[s,a,b]
//   (the last two of the chained mode-n products of the low-rank compression).
// back_tail (read+write W once): per slab, expand the two trailing modes of the
//   normalised core, D[s,a,b] = sum_{ja,jb} Ua[a,ja] Ub[b,jb] T'[s,ja,jb], and apply
//   W <- (1 - eta wd) W - eta alpha D, then W[Omega] -= eta lambda N_S
//   (reconstruction, scaled sparse add and weight update of Algorithm 1).
//
// Lane l of the warp owns rows a = l + 32 r of the slab (r < RPL); the rb
// columns of the small side live in registers (RBP = rb padded).
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

// Shared-memory layout (units of cf = 8 bytes; every region starts on 16 bytes):
//   [B][rbp] small factor | [A][ras] large factor | per warp: [A][Bs] slab, then the small tile
__host__ __device__ inline size_t tail_even(size_t x) { return (x + 1) & ~(size_t)1; }
__host__ __device__ inline size_t tail_warp_elems(int A, int Bs, int ra, int rbp, bool back) {
  return tail_even((size_t)A * Bs) + (back ? (size_t)ra * rbp : (size_t)A * rbp);
}
__host__ __device__ inline size_t tail_smem_bytes(int A, int B, int Bs, int ra, int ras, int rbp, int nwarps, bool back) {
  return 8 * ((size_t)B * rbp + tail_even((size_t)A * ras) + (size_t)nwarps * tail_warp_elems(A, Bs, ra, rbp, back));
}

template <class S, int RPL, int RBP>
__global__ void __launch_bounds__(256) proj_tail_kernel(const void* __restrict__ g, TailParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int nw = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int A = p.A, B = p.B, Bs = p.Bs, ra = p.ra, rb = p.rb, ras = p.ras;
  cf* ub_s = reinterpret_cast<cf*>(smem_raw);              // [B][RBP]   conj(Ub), zero padded
  cf* ua_s = ub_s + (size_t)B * RBP;                       // [A][ras]   conj(Ua)
  cf* xs = ua_s + tail_even((size_t)A * ras) + (size_t)warp * tail_warp_elems(A, Bs, ra, RBP, false);   // [A][Bs]
  cf* ys = xs + tail_even((size_t)A * Bs);                 // [A][RBP]

  for (int i = threadIdx.x; i < B * RBP; i += blockDim.x) {
    int b = i / RBP, j = i - b * RBP;
    cf u = (j < rb) ? p.Ub[b * rb + j] : make_float2(0.f, 0.f);
    ub_s[i] = make_float2(u.x, -u.y);
  }
  for (int i = threadIdx.x; i < A * ra; i += blockDim.x) {
    int a = i / ra, j = i - a * ra;
    cf u = p.Ua[i];
    ua_s[a * ras + j] = make_float2(u.x, -u.y);
  }
  __syncthreads();

  const uint32_t E = p.E;
  for (uint32_t s = blockIdx.x * nw + warp; s < p.nslab; s += gridDim.x * nw) {
    const size_t gbase = (size_t)s * E;
    // ---- slab -> shared (row stride Bs) ----
    if (Bs == B) {
      for (uint32_t i = lane; i < E; i += 32) xs[i] = S::load(g, gbase + i);
    } else {
      for (uint32_t i = lane; i < E; i += 32) { uint32_t a = i / B; xs[a * Bs + (i - a * B)] = S::load(g, gbase + i); }
    }
    __syncwarp();
    // ---- sparse part: gather, Adam, zero (residual) ----
    if (p.k > 0) {
      const int j0 = (int)p.slab_ptr[s], j1 = (int)p.slab_ptr[s + 1];
      for (int j = j0 + lane; j < j1; j += 32) {
        uint32_t loc = p.omega[j] - (uint32_t)gbase;
        uint32_t a = loc / B;
        uint32_t si = a * Bs + (loc - a * B);
        cf x = xs[si];
        xs[si] = make_float2(0.f, 0.f);
        cf m = p.m_s[j]; float v = p.v_s[j];
        cf n = adam_apply(x, m, v, p.adam);
        p.m_s[j] = m; p.v_s[j] = v; p.n_s[j] = n;
      }
      __syncwarp();
    }
    // ---- mode N:  Y[a][jb] = sum_b R[a][b] conj(Ub[b][jb]) ----
    for (int a0 = 0; a0 < A; a0 += 32 * RPL) {
      cf acc[RPL][RBP];
#pragma unroll
      for (int r = 0; r < RPL; ++r)
#pragma unroll
        for (int j = 0; j < RBP; ++j) acc[r][j] = make_float2(0.f, 0.f);
      int arow[RPL];
#pragma unroll
      for (int r = 0; r < RPL; ++r) { int a = a0 + lane + 32 * r; arow[r] = (a < A ? a : A - 1) * Bs; }
      for (int b = 0; b < B; ++b) {
        cf u[RBP];
        load_row_bcast<RBP>(ub_s + b * RBP, u);
#pragma unroll
        for (int r = 0; r < RPL; ++r) {
          cf x = xs[arow[r] + b];
#pragma unroll
          for (int j = 0; j < RBP; ++j) cfma(acc[r][j], x, u[j]);
        }
      }
#pragma unroll
      for (int r = 0; r < RPL; ++r) {
        int a = a0 + lane + 32 * r;
        if (a < A) {
#pragma unroll
          for (int j = 0; j < RBP; ++j) ys[a * RBP + j] = acc[r][j];
        }
      }
    }
    __syncwarp();
    // ---- mode N-1:  T[ja][jb] = sum_a conj(Ua[a][ja]) Y[a][jb];  4 consecutive jb per lane ----
    {
      constexpr int QJ = RBP / 4;
      const int ntask = ra * QJ;
      cf* tout = p.t + (size_t)s * ra * rb;
      for (int task = lane; task < ntask; task += 32) {
        int ja = task / QJ, jq = task - ja * QJ;
        cf acc[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j] = make_float2(0.f, 0.f);
        const cf* yp = ys + jq * 4;
        const cf* up = ua_s + ja;
        for (int a = 0; a < A; ++a) {
          cf u = up[a * ras];
          cf y[4];
          load_row_bcast<4>(yp + a * RBP, y);
#pragma unroll
          for (int j = 0; j < 4; ++j) cfma(acc[j], u, y[j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          int jb = jq * 4 + j;
          if (jb < rb) tout[ja * rb + jb] = acc[j];
        }
      }
    }
    __syncwarp();
  }
}

template <class S, int RPL, int RBP>
__global__ void __launch_bounds__(256) back_tail_kernel(void* __restrict__ w, TailParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int nw = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int A = p.A, B = p.B, Bs = p.Bs, ra = p.ra, rb = p.rb, ras = p.ras;
  cf* ub_s = reinterpret_cast<cf*>(smem_raw);              // [B][RBP]  Ub, zero padded
  cf* ua_s = ub_s + (size_t)B * RBP;                       // [A][ras]  Ua
  cf* ws = ua_s + tail_even((size_t)A * ras) + (size_t)warp * tail_warp_elems(A, Bs, ra, RBP, true);    // [A][Bs]
  cf* ts = ws + tail_even((size_t)A * Bs);                 // [ra][RBP]

  for (int i = threadIdx.x; i < B * RBP; i += blockDim.x) {
    int b = i / RBP, j = i - b * RBP;
    ub_s[i] = (j < rb) ? p.Ub[b * rb + j] : make_float2(0.f, 0.f);
  }
  for (int i = threadIdx.x; i < A * ra; i += blockDim.x) {
    int a = i / ra, j = i - a * ra;
    ua_s[a * ras + j] = p.Ua[i];
  }
  __syncthreads();

  const uint32_t E = p.E;
  const bool decay = p.decay != 1.0f;
  for (uint32_t s = blockIdx.x * nw + warp; s < p.nslab; s += gridDim.x * nw) {
    const size_t gbase = (size_t)s * E;
    // ---- W slab and T' tile -> shared ----
    if (Bs == B) {
      for (uint32_t i = lane; i < E; i += 32) ws[i] = S::load(w, gbase + i);
    } else {
      for (uint32_t i = lane; i < E; i += 32) { uint32_t a = i / B; ws[a * Bs + (i - a * B)] = S::load(w, gbase + i); }
    }
    {
      const cf* tin = p.t + (size_t)s * ra * rb;
      for (int i = lane; i < ra * RBP; i += 32) {
        int ja = i / RBP, j = i - ja * RBP;
        ts[i] = (j < rb) ? tin[ja * rb + j] : make_float2(0.f, 0.f);
      }
    }
    __syncwarp();
    for (int a0 = 0; a0 < A; a0 += 32 * RPL) {
      // ---- mode N-1:  Y'[a][jb] = sum_ja Ua[a][ja] T'[ja][jb] ----
      cf y[RPL][RBP];
#pragma unroll
      for (int r = 0; r < RPL; ++r)
#pragma unroll
        for (int j = 0; j < RBP; ++j) y[r][j] = make_float2(0.f, 0.f);
      int urow[RPL], wrow[RPL];
      bool ok[RPL];
#pragma unroll
      for (int r = 0; r < RPL; ++r) {
        int a = a0 + lane + 32 * r;
        ok[r] = a < A;
        int ac = ok[r] ? a : A - 1;
        urow[r] = ac * ras; wrow[r] = ac * Bs;
      }
      for (int ja = 0; ja < ra; ++ja) {
        cf tv[RBP];
        load_row_bcast<RBP>(ts + ja * RBP, tv);
#pragma unroll
        for (int r = 0; r < RPL; ++r) {
          cf u = ua_s[urow[r] + ja];
#pragma unroll
          for (int j = 0; j < RBP; ++j) cfma(y[r][j], u, tv[j]);
        }
      }
      // ---- mode N:  D[a][b] = sum_jb Y'[a][jb] Ub[b][jb];  W <- decay*W - eta*alpha*D ----
      for (int b = 0; b < B; ++b) {
        cf u[RBP];
        load_row_bcast<RBP>(ub_s + b * RBP, u);
#pragma unroll
        for (int r = 0; r < RPL; ++r) {
          cf d = make_float2(0.f, 0.f);
#pragma unroll
          for (int j = 0; j < RBP; ++j) cfma(d, y[r][j], u[j]);
          if (ok[r]) {
            cf wv = ws[wrow[r] + b];
            if (decay) { wv.x *= p.decay; wv.y *= p.decay; }
            wv.x = fmaf(-p.s_low, d.x, wv.x);
            wv.y = fmaf(-p.s_low, d.y, wv.y);
            ws[wrow[r] + b] = wv;
          }
        }
      }
    }
    __syncwarp();
    // ---- scaled sparse add at Omega (on top of the dense update) ----
    if (p.k > 0) {
      const int j0 = (int)p.slab_ptr[s], j1 = (int)p.slab_ptr[s + 1];
      for (int j = j0 + lane; j < j1; j += 32) {
        uint32_t loc = p.omega[j] - (uint32_t)gbase;
        uint32_t a = loc / B;
        uint32_t si = a * Bs + (loc - a * B);
        cf wv = ws[si];
        if (S::kBytes == 4) {   // half storage: the dense update is rounded to fp16 before the sparse add
          wv = __half22float2(__floats2half2_rn(wv.x, wv.y));
        }
        cf n = p.n_s[j];
        wv.x = fmaf(-p.s_sparse, n.x, wv.x);
        wv.y = fmaf(-p.s_sparse, n.y, wv.y);
        ws[si] = wv;
      }
      __syncwarp();
    }
    if (Bs == B) {
      for (uint32_t i = lane; i < E; i += 32) S::store(w, gbase + i, ws[i]);
    } else {
      for (uint32_t i = lane; i < E; i += 32) { uint32_t a = i / B; S::store(w, gbase + i, ws[a * Bs + (i - a * B)]); }
    }
    __syncwarp();
  }
}

}  // namespace tg
