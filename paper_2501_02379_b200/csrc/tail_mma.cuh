// Fast path of the two streaming kernels: slabs arrive by bulk asynchronous copy
// into a per-warp ring in shared memory, and the two trailing mode products run
// on the tensor cores as split-precision TF32 (x = hi + lo, three products, fp32
// accumulation), chained through registers: the accumulator fragments of the
// first product are the operand fragments of the second.
//
// Complex arithmetic is carried as real arithmetic on interleaved (re, im) data:
//   Y = X conj(Ub):  [Yre; Yim] = W1 [Xre; Xim],  W1 = [[ur, ui], [-ui, ur]]
//   T = conj(Ua)^T Y:[Tre; Tim] = W2 [Yre; Yim],  W2 = [[ur, ui], [-ui, ur]]
// and without conjugation for the reconstruction.
//
// proj (compression, trailing modes N then N-1), per slab X[A][B]:
//   stage 1  D1[(c,jb)][a] = sum_{(b,c')} W1[(c,jb)][(b,c')] X[a][(b,c')]      m16 = (re|im) x 8 jb, n8 = 8 rows a
//   stage 2  D2[(c,ja)][jb] = sum_{(a,c')} W2[(c,ja)][(a,c')] Y[(a,c')][jb]    m16 = (re|im) x 8 ja, n8 = 8 jb
// The K index inside one MMA step is a free permutation as long as both
// operands use the same one; it is chosen so that every operand load is one
// conflict-free 8-byte shared-memory access:
//   stage 1, step (kb, j): k = t <-> (b, re), k = t+4 <-> (b, im), b = 16 kb + 4 t + j
//   stage 2, step (nt, c): k = t <-> (a, c),  k = t+4 <-> (a+1, c), a = a0 + 8 nt + 2 t
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "tail.cuh"

namespace tg {

struct TailMmaGeom {
  int nwarps, nbuf;          // warps per block, ring depth per warp
  int rbs, ras;              // padded row lengths (complex) of the small / large factor copies in shared memory
  uint32_t slab_bytes;       // E * 8
  uint32_t buf_stride;       // bytes between ring buffers (slab_bytes rounded up to 128)
  uint32_t off_ua, off_ring, off_bar, total;   // byte offsets in dynamic shared memory
};

__host__ __device__ inline int tm_rbs(int rbt) { return 8 * rbt + 2; }                                  // == 2 (mod 4)
__host__ __device__ inline int tm_ras(int rat) { return 8 * rat + 4; }                                  // == 4 (mod 8)

__host__ inline TailMmaGeom tail_mma_geom(int A, int B, int rat, int rbt, int nwarps, int nbuf) {
  TailMmaGeom g;
  g.nwarps = nwarps; g.nbuf = nbuf;
  g.rbs = tm_rbs(rbt); g.ras = tm_ras(rat);
  g.slab_bytes = (uint32_t)A * B * 8;
  g.buf_stride = (g.slab_bytes + 127) & ~127u;
  uint32_t ub = (uint32_t)B * g.rbs * 8 * 2;            // hi and lo copies
  uint32_t ua = (uint32_t)A * g.ras * 8;                // raw copy, split on the fly
  g.off_ua = (ub + 127) & ~127u;
  g.off_ring = (g.off_ua + ua + 127) & ~127u;
  g.off_bar = g.off_ring + (uint32_t)nwarps * nbuf * g.buf_stride;
  g.total = g.off_bar + (uint32_t)nwarps * nbuf * 8;
  return g;
}

struct TailMmaParams {
  TailParams p;
  TailMmaGeom g;
  int* flags;      // sticky status word (bit 4: a bulk copy did not arrive within the wait limit)
};

__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) { hi = tf32_hi(x); lo = x - hi; }

// All lanes wait (bounded) for a phase of the barrier and agree on the outcome.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) {
  bool ok = mbar_wait_bounded(bar, parity);
  if (!__all_sync(0xffffffffu, ok)) {        // a lane ran out of polls just as the phase completed
    ok = mbar_try_wait(bar, parity);
    ok = __all_sync(0xffffffffu, ok);
  }
  return ok;
}

// Copies the factor matrices into shared memory, zero padded: the small one as (hi, lo) TF32 pairs,
// the large one as it is (split when used).
__device__ __forceinline__ void stage_factors(unsigned char* smem, const TailMmaParams& P) {
  const TailParams& p = P.p;
  const int rbs = P.g.rbs, ras = P.g.ras;
  cf* ubh = reinterpret_cast<cf*>(smem);
  cf* ubl = ubh + (size_t)p.B * rbs;
  cf* uas = reinterpret_cast<cf*>(smem + P.g.off_ua);
  for (int i = threadIdx.x; i < p.B * rbs; i += blockDim.x) {
    int b = i / rbs, j = i - b * rbs;
    cf u = (j < p.rb) ? p.Ub[b * p.rb + j] : make_float2(0.f, 0.f);
    cf h, l; split_tf32(u.x, h.x, l.x); split_tf32(u.y, h.y, l.y);
    ubh[i] = h; ubl[i] = l;
  }
  for (int i = threadIdx.x; i < p.A * ras; i += blockDim.x) {
    int a = i / ras, j = i - a * ras;
    uas[i] = (j < p.ra) ? p.Ua[a * p.ra + j] : make_float2(0.f, 0.f);
  }
}

// ---------------------------------------------------------------------------------------------
// Compression of the two trailing modes, fused with the sparse gather / Adam / residual.
// RAT = ceil(ra/8), RBT = ceil(rb/8), NT = row tiles (of 8) handled per pass, A % (8 NT) == 0.
// ---------------------------------------------------------------------------------------------
template <int RAT, int RBT, int NT>
__global__ void __launch_bounds__(256) proj_tail_mma_kernel(const void* __restrict__ g, TailMmaParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  const TailParams& p = P.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, t = lane & 3;
  const int A = p.A, B = p.B, ra = p.ra, rb = p.rb, rbs = P.g.rbs, ras = P.g.ras, nbuf = P.g.nbuf;
  const int twoB = 2 * B;
  const cf* ubh = reinterpret_cast<const cf*>(smem);
  const cf* ubl = ubh + (size_t)B * rbs;
  const cf* uas = reinterpret_cast<const cf*>(smem + P.g.off_ua);
  unsigned char* ring = smem + P.g.off_ring + (size_t)warp * nbuf * P.g.buf_stride;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P.g.off_bar) + warp * nbuf;

  stage_factors(smem, P);
  if (lane == 0)
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
  fence_mbar_init();
  __syncthreads();

  const uint32_t E = p.E, nslab = p.nslab;
  const uint32_t wstride = gridDim.x * P.g.nwarps;
  const uint32_t s_first = blockIdx.x * P.g.nwarps + warp;
  const unsigned char* gb = static_cast<const unsigned char*>(g);
  // prologue: fill the ring
  if (lane == 0) {
    uint32_t s = s_first;
    for (int i = 0; i < nbuf - 1 && s < nslab; ++i, s += wstride) {
      mbar_expect_tx(&bars[i], P.g.slab_bytes);
      bulk_g2s(ring + (size_t)i * P.g.buf_stride, gb + (size_t)s * P.g.slab_bytes, P.g.slab_bytes, &bars[i]);
    }
  }
  const int KB = twoB / 32, rem = twoB - 32 * KB;
  const int KS1 = 4 * KB + (rem >= 8 ? 4 : rem / 2);   // steps of the last block in which lane t = 0 is still inside the row
  uint32_t it = 0;
  for (uint32_t s = s_first; s < nslab; s += wstride, ++it) {
    const int buf = it % nbuf;
    // keep the ring full: the buffer freed by the previous iteration takes the slab nbuf-1 ahead
    if (lane == 0) {
      uint32_t sn = s + (uint32_t)(nbuf - 1) * wstride;
      if (sn < nslab) {
        int bn = (it + nbuf - 1) % nbuf;
        fence_async_smem();   // the buffer was last written through the generic proxy (zeroed sparse entries)
        mbar_expect_tx(&bars[bn], P.g.slab_bytes);
        bulk_g2s(ring + (size_t)bn * P.g.buf_stride, gb + (size_t)sn * P.g.slab_bytes, P.g.slab_bytes, &bars[bn]);
      }
    }
    if (!warp_wait(&bars[buf], (it / nbuf) & 1)) {
      // give up: record it, drain whatever else this warp still has in flight (bounded), leave
      if (lane == 0) atomicOr(P.flags, 4);
      for (int i = 1; i < nbuf; ++i)
        if (s + (uint32_t)i * wstride < nslab) mbar_wait_bounded(&bars[(it + i) % nbuf], ((it + i) / nbuf) & 1, 1u << 16);
      break;
    }
    float* xs = reinterpret_cast<float*>(ring + (size_t)buf * P.g.buf_stride);
    const size_t gbase = (size_t)s * E;
    // ---- sparse part: gather, Adam, zero (residual) ----
    if (p.k > 0) {
      const int j0 = (int)p.slab_ptr[s], j1 = (int)p.slab_ptr[s + 1];
      for (int j = j0 + lane; j < j1; j += 32) {
        uint32_t loc = p.omega[j] - (uint32_t)gbase;
        cf* xp = reinterpret_cast<cf*>(xs) + loc;
        cf x = *xp;
        *xp = make_float2(0.f, 0.f);
        cf m = p.m_s[j]; float v = p.v_s[j];
        cf n = adam_apply(x, m, v, p.adam);
        p.m_s[j] = m; p.v_s[j] = v; p.n_s[j] = n;
      }
      __syncwarp();
    }
    float d2[RAT][RBT][4];
#pragma unroll
    for (int mt = 0; mt < RAT; ++mt)
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
        for (int i = 0; i < 4; ++i) d2[mt][jt][i] = 0.f;

    for (int a0 = 0; a0 < A; a0 += 8 * NT) {
      float d1[RBT][NT][4];
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) d1[jt][nt][i] = 0.f;
      // ---- stage 1 ----
      const float* xrow = xs + (size_t)(a0 + gq) * twoB;
      for (int ks = 0; ks < KS1; ++ks) {
        const int f = 32 * (ks >> 2) + 8 * t + 2 * (ks & 3);    // float index inside the row (even)
        const bool valid = f < twoB;
        const int b = f >> 1;
        cf uh[RBT], ul[RBT];
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          uh[jt] = valid ? ubh[b * rbs + 8 * jt + gq] : make_float2(0.f, 0.f);
          ul[jt] = valid ? ubl[b * rbs + 8 * jt + gq] : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float2 x = valid ? *reinterpret_cast<const float2*>(xrow + (size_t)nt * 8 * twoB + f) : make_float2(0.f, 0.f);
          float xh0, xl0, xh1, xl1;
          split_tf32(x.x, xh0, xl0); split_tf32(x.y, xh1, xl1);
#pragma unroll
          for (int jt = 0; jt < RBT; ++jt) {
            mma_tf32(d1[jt][nt], uh[jt].x, -uh[jt].y, uh[jt].y, uh[jt].x, xh0, xh1);
            mma_tf32(d1[jt][nt], ul[jt].x, -ul[jt].y, ul[jt].y, ul[jt].x, xh0, xh1);
            mma_tf32(d1[jt][nt], uh[jt].x, -uh[jt].y, uh[jt].y, uh[jt].x, xl0, xl1);
          }
        }
      }
      // ---- stage 2: the accumulators of stage 1 are the B fragments ----
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int a = a0 + 8 * nt + 2 * t;
        float yh[RBT][4], yl[RBT][4];
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
          for (int i = 0; i < 4; ++i) split_tf32(d1[jt][nt][i], yh[jt][i], yl[jt][i]);
#pragma unroll
        for (int mt = 0; mt < RAT; ++mt) {
          const int ja = 8 * mt + gq;
          const cf u0 = uas[a * ras + ja], u1 = uas[(a + 1) * ras + ja];
          cf u0h, u0l, u1h, u1l;
          split_tf32(u0.x, u0h.x, u0l.x); split_tf32(u0.y, u0h.y, u0l.y);
          split_tf32(u1.x, u1h.x, u1l.x); split_tf32(u1.y, u1h.y, u1l.y);
#pragma unroll
          for (int jt = 0; jt < RBT; ++jt) {
            // k-step (nt, re): B = (Yre[a], Yre[a+1])
            mma_tf32(d2[mt][jt], u0h.x, -u0h.y, u1h.x, -u1h.y, yh[jt][0], yh[jt][1]);
            mma_tf32(d2[mt][jt], u0l.x, -u0l.y, u1l.x, -u1l.y, yh[jt][0], yh[jt][1]);
            mma_tf32(d2[mt][jt], u0h.x, -u0h.y, u1h.x, -u1h.y, yl[jt][0], yl[jt][1]);
            // k-step (nt, im): B = (Yim[a], Yim[a+1])
            mma_tf32(d2[mt][jt], u0h.y, u0h.x, u1h.y, u1h.x, yh[jt][2], yh[jt][3]);
            mma_tf32(d2[mt][jt], u0l.y, u0l.x, u1l.y, u1l.x, yh[jt][2], yh[jt][3]);
            mma_tf32(d2[mt][jt], u0h.y, u0h.x, u1h.y, u1h.x, yl[jt][2], yl[jt][3]);
          }
        }
      }
    }
    // ---- T[s][ja][jb]: d0 = Tre[ja][jb], d1 = Tre[ja][jb+1], d2 = Tim[ja][jb], d3 = Tim[ja][jb+1] ----
    cf* tout = p.t + (size_t)s * ra * rb;
#pragma unroll
    for (int mt = 0; mt < RAT; ++mt) {
      const int ja = 8 * mt + gq;
      if (ja >= ra) continue;
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt) {
        const int jb = 8 * jt + 2 * t;
        const float* d = d2[mt][jt];
        if ((rb & 1) == 0 && jb + 1 < rb) {
          *reinterpret_cast<float4*>(tout + (size_t)ja * rb + jb) = make_float4(d[0], d[2], d[1], d[3]);
        } else {
          if (jb < rb) tout[(size_t)ja * rb + jb] = make_float2(d[0], d[2]);
          if (jb + 1 < rb) tout[(size_t)ja * rb + jb + 1] = make_float2(d[1], d[3]);
        }
      }
    }
    __syncwarp();   // every lane is done with this buffer before lane 0 refills it
  }
}

// ---------------------------------------------------------------------------------------------
// Reconstruction of the two trailing modes, fused with the weight update and the sparse add.
// Per slab W[A][B], with T'[ra][rb] the slab's tile of the partly reconstructed core:
//   stage 1  D1[a][(c,jb)] = sum_{(ja,c')} Ua[a][(ja,c')] Tt[(ja,c')][(c,jb)]     m16 = 16 rows a, n8 = (re|im) x 8 jb
//   stage 2  D [a][(b,c)]  = sum_{(jb,c')} Y'[a][(jb,c')] W3[(jb,c')][(b,c)]      m16 = 16 rows a, n8 = 4 complex b
// stage 1, step ks: k = t <-> (ja, re), k = t+4 <-> (ja, im), ja = 4 ks + t
// stage 2, step (c', jt): k = t <-> (jb, c'), k = t+4 <-> (jb+1, c'), jb = 8 jt + 2 t  (the accumulator layout of stage 1)
// stage 2, tile (kb, j): n = g <-> (b, g & 1), b = 16 kb + 4 (g >> 1) + j, so that lane (g, t) owns W[a][16 kb + 4 t + j]
// ---------------------------------------------------------------------------------------------
template <int RAT, int RBT>
__global__ void __launch_bounds__(256) back_tail_mma_kernel(void* __restrict__ w, TailMmaParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  const TailParams& p = P.p;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, t = lane & 3;
  const int A = p.A, B = p.B, ra = p.ra, rb = p.rb, rbs = P.g.rbs, ras = P.g.ras, nbuf = P.g.nbuf;
  const int twoB = 2 * B;
  const cf* ubh = reinterpret_cast<const cf*>(smem);
  const cf* ubl = ubh + (size_t)B * rbs;
  const cf* uas = reinterpret_cast<const cf*>(smem + P.g.off_ua);
  unsigned char* ring = smem + P.g.off_ring + (size_t)warp * nbuf * P.g.buf_stride;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P.g.off_bar) + warp * nbuf;

  stage_factors(smem, P);
  if (lane == 0)
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
  fence_mbar_init();
  __syncthreads();

  const uint32_t E = p.E, nslab = p.nslab;
  const uint32_t wstride = gridDim.x * P.g.nwarps;
  const uint32_t s_first = blockIdx.x * P.g.nwarps + warp;
  unsigned char* wb = static_cast<unsigned char*>(w);
  // The ring is filled nbuf-2 slabs ahead: the buffer stored at iteration it-1 may still be read by
  // its bulk store while iteration it runs, so the refill at iteration it goes to the buffer of it-2.
  const int dist = nbuf - 2 > 0 ? nbuf - 2 : 0;
  if (lane == 0) {
    uint32_t s = s_first;
    for (int i = 0; i < dist && s < nslab; ++i, s += wstride) {
      mbar_expect_tx(&bars[i], P.g.slab_bytes);
      bulk_g2s(ring + (size_t)i * P.g.buf_stride, wb + (size_t)s * P.g.slab_bytes, P.g.slab_bytes, &bars[i]);
    }
  }
  const int KB = twoB / 32, rem = twoB - 32 * KB;
  const int NB = 4 * KB + (rem >= 8 ? 4 : rem / 2);   // column tiles (4 complex each) that hold any b < B
  constexpr int KS2 = 2 * RAT;                         // steps of 4 ja
  const bool decay = p.decay != 1.0f;
  uint32_t it = 0;
  bool failed = false;
  for (uint32_t s = s_first; s < nslab; s += wstride, ++it) {
    const int buf = it % nbuf;
    if (lane == 0) {
      uint32_t sn = s + (uint32_t)dist * wstride;
      if (sn < nslab) {
        int bn = (it + dist) % nbuf;
        bulk_wait_read<1>();          // every bulk store but the newest has finished reading its buffer
        mbar_expect_tx(&bars[bn], P.g.slab_bytes);
        bulk_g2s(ring + (size_t)bn * P.g.buf_stride, wb + (size_t)sn * P.g.slab_bytes, P.g.slab_bytes, &bars[bn]);
      }
    }
    // T' fragments for stage 1 (read while the slab is in flight): T'[ja = 4 ks + t][jb = 8 jt + g]
    float tbh[KS2][RBT][2], tbl[KS2][RBT][2];
    {
      const cf* tin = p.t + (size_t)s * ra * rb;
#pragma unroll
      for (int ks = 0; ks < KS2; ++ks)
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          const int ja = 4 * ks + t, jb = 8 * jt + gq;
          cf v = (ja < ra && jb < rb) ? __ldg(tin + (size_t)ja * rb + jb) : make_float2(0.f, 0.f);
          split_tf32(v.x, tbh[ks][jt][0], tbl[ks][jt][0]);
          split_tf32(v.y, tbh[ks][jt][1], tbl[ks][jt][1]);
        }
    }
    if (!warp_wait(&bars[buf], (it / nbuf) & 1)) {
      if (lane == 0) atomicOr(P.flags, 4);
      for (int i = 1; i <= dist; ++i)
        if (s + (uint32_t)i * wstride < nslab) mbar_wait_bounded(&bars[(it + i) % nbuf], ((it + i) / nbuf) & 1, 1u << 16);
      failed = true;
      break;
    }
    float* ws = reinterpret_cast<float*>(ring + (size_t)buf * P.g.buf_stride);
    const size_t gbase = (size_t)s * E;

    for (int am = 0; am < A; am += 16) {
      // ---- stage 1: Y'[a][(c, jb)] for rows am+g and am+g+8 ----
      float d1[2][RBT][4];
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
          for (int i = 0; i < 4; ++i) d1[c][jt][i] = 0.f;
      const int r0 = am + gq, r1 = (am + gq + 8 < A) ? am + gq + 8 : r0;   // r1 clamps when A % 16 == 8
      const bool r1ok = am + gq + 8 < A;
#pragma unroll
      for (int ks = 0; ks < KS2; ++ks) {
        const int ja = 4 * ks + t;
        const cf u0 = uas[r0 * ras + ja], u1 = uas[r1 * ras + ja];
        cf u0h, u0l, u1h, u1l;
        split_tf32(u0.x, u0h.x, u0l.x); split_tf32(u0.y, u0h.y, u0l.y);
        split_tf32(u1.x, u1h.x, u1l.x); split_tf32(u1.y, u1h.y, u1l.y);
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          const float trh = tbh[ks][jt][0], tih = tbh[ks][jt][1], trl = tbl[ks][jt][0], til = tbl[ks][jt][1];
          // A = (Ua[r0].re, Ua[r1].re, Ua[r0].im, Ua[r1].im);  re tile: B = (Tr, -Ti);  im tile: B = (Ti, Tr)
          mma_tf32(d1[0][jt], u0h.x, u1h.x, u0h.y, u1h.y, trh, -tih);
          mma_tf32(d1[0][jt], u0l.x, u1l.x, u0l.y, u1l.y, trh, -tih);
          mma_tf32(d1[0][jt], u0h.x, u1h.x, u0h.y, u1h.y, trl, -til);
          mma_tf32(d1[1][jt], u0h.x, u1h.x, u0h.y, u1h.y, tih, trh);
          mma_tf32(d1[1][jt], u0l.x, u1l.x, u0l.y, u1l.y, tih, trh);
          mma_tf32(d1[1][jt], u0h.x, u1h.x, u0h.y, u1h.y, til, trl);
        }
      }
      // split Y' once: a0 = d[0] (row g, jb), a1 = d[2] (row g+8, jb), a2 = d[1] (row g, jb+1), a3 = d[3]
      float yh[2][RBT][4], yl[2][RBT][4];
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
          for (int i = 0; i < 4; ++i) split_tf32(d1[c][jt][i], yh[c][jt][i], yl[c][jt][i]);
      // ---- stage 2, one column tile at a time, applied to the slab right away ----
      for (int nb = 0; nb < NB; ++nb) {
        const int colbase = 16 * (nb >> 2) + (nb & 3);
        const int bq = colbase + 4 * (gq >> 1);          // the b this lane supplies as operand column n = g
        const bool bq_ok = bq < B;
        const bool odd = gq & 1;                         // n odd <-> imaginary output component
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          // Ub[bq][jb], Ub[bq][jb+1] with jb = 8 jt + 2 t  (rbs is even, so the pair is 16-byte aligned)
          float4 qh = bq_ok ? *reinterpret_cast<const float4*>(ubh + (size_t)bq * rbs + 8 * jt + 2 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
          float4 ql = bq_ok ? *reinterpret_cast<const float4*>(ubl + (size_t)bq * rbs + 8 * jt + 2 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
          // step c' = re: W3[(jb,re)][(b,re)] = ur, [(b,im)] = ui;  step c' = im: [(b,re)] = -ui, [(b,im)] = ur
          const float b0re_h = odd ? qh.y : qh.x, b1re_h = odd ? qh.w : qh.z;
          const float b0re_l = odd ? ql.y : ql.x, b1re_l = odd ? ql.w : ql.z;
          const float b0im_h = odd ? qh.x : -qh.y, b1im_h = odd ? qh.z : -qh.w;
          const float b0im_l = odd ? ql.x : -ql.y, b1im_l = odd ? ql.z : -ql.w;
          mma_tf32(d, yh[0][jt][0], yh[0][jt][2], yh[0][jt][1], yh[0][jt][3], b0re_h, b1re_h);
          mma_tf32(d, yl[0][jt][0], yl[0][jt][2], yl[0][jt][1], yl[0][jt][3], b0re_h, b1re_h);
          mma_tf32(d, yh[0][jt][0], yh[0][jt][2], yh[0][jt][1], yh[0][jt][3], b0re_l, b1re_l);
          mma_tf32(d, yh[1][jt][0], yh[1][jt][2], yh[1][jt][1], yh[1][jt][3], b0im_h, b1im_h);
          mma_tf32(d, yl[1][jt][0], yl[1][jt][2], yl[1][jt][1], yl[1][jt][3], b0im_h, b1im_h);
          mma_tf32(d, yh[1][jt][0], yh[1][jt][2], yh[1][jt][1], yh[1][jt][3], b0im_l, b1im_l);
        }
        // d0 + i d1 = D[row g][b], d2 + i d3 = D[row g+8][b] with b = colbase + 4 t
        const int bo = colbase + 4 * t;
        if (bo < B) {
          float2* w0 = reinterpret_cast<float2*>(ws + (size_t)r0 * twoB) + bo;
          float2 v0 = *w0;
          if (decay) { v0.x *= p.decay; v0.y *= p.decay; }
          v0.x = fmaf(-p.s_low, d[0], v0.x); v0.y = fmaf(-p.s_low, d[1], v0.y);
          *w0 = v0;
          if (r1ok) {
            float2* w1 = reinterpret_cast<float2*>(ws + (size_t)r1 * twoB) + bo;
            float2 v1 = *w1;
            if (decay) { v1.x *= p.decay; v1.y *= p.decay; }
            v1.x = fmaf(-p.s_low, d[2], v1.x); v1.y = fmaf(-p.s_low, d[3], v1.y);
            *w1 = v1;
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
        cf* wp = reinterpret_cast<cf*>(ws) + loc;
        cf wv = *wp;
        cf n = p.n_s[j];
        wv.x = fmaf(-p.s_sparse, n.x, wv.x);
        wv.y = fmaf(-p.s_sparse, n.y, wv.y);
        *wp = wv;
      }
    }
    fence_async_smem();     // order this lane's shared-memory writes before the bulk store reads them
    __syncwarp();
    if (lane == 0) {
      bulk_s2g(wb + (size_t)s * P.g.slab_bytes, ws, P.g.slab_bytes);
      bulk_commit();
    }
  }
  if (lane == 0 && !failed) bulk_wait_all<0>();   // stores complete before the block's shared memory goes away
}

}  // namespace tg
