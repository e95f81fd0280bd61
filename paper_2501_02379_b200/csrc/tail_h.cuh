// Streaming kernels for half-precision storage (W and G as interleaved fp16 pairs; the mixed-precision
// recipe of Section 2.3) and slabs of up to 128 rows.
//
// A slab arrives by one bulk asynchronous copy as it is stored (fp16), and stays fp16 in shared memory.
// fp16 values are exact fp16 MMA operands, so the first trailing-mode product needs no splitting of the
// streamed operand at all: Y = X conj(Ub) is two m16n8k16 MMAs per step (Ub = hi + lo in fp16, X exact),
// at twice the K per instruction of the TF32 shape.  The second product of the compression (over the slab rows, whose
// operand carries the gradient's scale) runs as split-precision TF32 like the fp32-storage kernels; the two products
// of the reconstruction run as fp16 MMAs on two-term splits (see back_tail_h_kernel).
//
// A block has one warp per tile of 8 slab rows (A/8 warps, at most 16) and works on one slab at a time
// from a ring of bulk copies; one block per SM.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "tail.cuh"
#include "tail_tc.cuh"

namespace tg {

struct TailHGeom {
  int nwarps, nbuf, ks16;      // warps (= row tiles of 8), ring depth, k16-steps of the first product (8 columns b each)
  int ldy, ldu;                // row lengths (complex) of the Y and Ua copies in shared memory
  int ntile2, ksplit;          // second product: (m, n) output tiles, and how many warps share one tile's K range
  uint32_t slab_bytes, buf_stride;
  uint32_t off_u1, off_ua, off_y, off_part, off_bar, total;
};

__host__ inline bool tail_h_geom(int A, int B, int ra, int rb, TailHGeom& g) {
  if (A % 8 || A < 8 || A > 128) return false;
  const int rat = (ra + 7) / 8, rbt = (rb + 7) / 8;
  if (rat > 4 || rbt > 2) return false;
  g.nwarps = A / 8;
  g.ks16 = 4 * (B / 32) + ((B % 32) < 4 ? (B % 32) : 4);     // see the column mapping of the first product
  g.ldy = 8 * rbt + 4; g.ldu = 8 * rat + 4;
  g.ntile2 = rat * rbt;
  g.ksplit = g.nwarps >= g.ntile2 ? g.nwarps / g.ntile2 : 1;
  if ((A / 4) % g.ksplit) return false;
  g.slab_bytes = (uint32_t)A * B * 4;
  if (g.slab_bytes % 16) return false;
  g.buf_stride = (g.slab_bytes + 127) & ~127u;
  const uint32_t u1 = (uint32_t)g.ks16 * rbt * 2 * 32 * 16;              // (hi, lo) x 4 registers per lane
  const uint32_t ua = (uint32_t)A * g.ldu * 8;
  const uint32_t y = 2u * A * g.ldy * 8;                                  // two stages
  const uint32_t units = (uint32_t)g.ntile2 * g.ksplit;
  const uint32_t part = 2u * units * 128 * 4;                             // two stages of partial tiles
  const uint32_t fixed = u1 + ua + y + part + 256;
  if (fixed + 2 * g.buf_stride > 227u * 1024u) return false;
  int nbuf = (int)((227u * 1024u - fixed) / g.buf_stride);
  if (nbuf > 4) nbuf = 4;
  g.nbuf = nbuf;
  g.off_u1 = (uint32_t)nbuf * g.buf_stride;
  g.off_ua = g.off_u1 + u1;
  g.off_y = g.off_ua + ua;
  g.off_part = g.off_y + y;
  g.off_bar = g.off_part + part;
  g.total = g.off_bar + 256;
  return true;
}

struct TailHParams {
  TailParams p;
  TailHGeom g;
  int* flags;
};

__device__ __forceinline__ uint32_t h2_bits(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }

// x = hi + lo in fp16 (|x| <= 1: the factor matrices have orthonormal columns)
__device__ __forceinline__ void split_f16(float x, __half& hi, __half& lo) {
  hi = __float2half_rn(x);
  lo = __float2half_rn(x - __half2float(hi));
}

// x = hi + lo / 2048 with hi, lo in fp16: lo carries the 11 bits below hi's at hi's own scale, so that neither part
// nears the subnormal range before x itself does.
constexpr float kF16LoScale = 2048.f, kF16LoInv = 1.f / 2048.f;
__device__ __forceinline__ void split_f16_scaled(float x, __half& hi, __half& lo) {
  hi = __float2half_rn(x);
  lo = __float2half_rn((x - __half2float(hi)) * kF16LoScale);
}

// ---------------------------------------------------------------------------------------------
// Compression of the two trailing modes (half storage), fused with the sparse gather and the residual.
//   stage 1 (fp16 m16n8k16), warp = tile of 8 rows a:
//     D1[(c,jb)][a] = sum_{(b,c')} W1[(c,jb)][(b,c')] X[a][(b,c')],  W1 rows (re,jb): (ur, ui), rows (im,jb): (-ui, ur)
//     step ks = (kb, jj): k = 2t, 2t+1 <-> (b1, re|im), k = 2t+8, 2t+9 <-> (b2, re|im), b1 = 32 kb + 8 t + jj, b2 = b1 + 4
//     (lanes of a quad read columns 8 apart: with rows of 65 words, all 32 loads of a step hit distinct banks)
//   stage 2 (split TF32 m16n8k8), block-wide: T'[(c,ja)][jb] = sum_{(a,c')} W2[(c,ja)][(a,c')] Y[(a,c')][jb];
//     a warp owns output tile (mt, nt) over one share of the rows a; step: k = t <-> (a, re), k = t+4 <-> (a, im), a = 4 q + t
// Software pipeline over the slabs of a block: iteration `it` runs stage 1 of slab it, stage 2 of slab it-1
// and the final sum of slab it-2, with one block-wide barrier.
// ---------------------------------------------------------------------------------------------
template <int RAT, int RBT>
__global__ void __launch_bounds__(512, 1) proj_tail_h_kernel(const void* __restrict__ g, TailHParams P) {
  griddep_chain();
  extern __shared__ __align__(128) unsigned char smem[];
  const TailParams& p = P.p;
  const TailHGeom& G = P.g;
  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  const int A = p.A, B = p.B, ra = p.ra, rb = p.rb, nbuf = G.nbuf, ldy = G.ldy, ldu = G.ldu, nwarps = G.nwarps;
  const int ks16 = G.ks16, ksplit = G.ksplit, units = G.ntile2 * G.ksplit;
  const uint32_t E = p.E, nslab = p.nslab, gstride = gridDim.x;
  uint4* u1tab = reinterpret_cast<uint4*>(smem + G.off_u1);       // [ks16][RBT][hi|lo][32]
  cf* uas = reinterpret_cast<cf*>(smem + G.off_ua);               // [A][ldu]
  cf* ysb = reinterpret_cast<cf*>(smem + G.off_y);                // [2][A][ldy]
  float* part = reinterpret_cast<float*>(smem + G.off_part);      // [2][units][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G.off_bar);
  const unsigned char* gb = static_cast<const unsigned char*>(g);

  // ---- Ub as stage-1 A fragments ----
  for (int idx = tid; idx < ks16 * RBT * 32; idx += nthr) {
    const int ks = idx / (RBT * 32), rem = idx - ks * (RBT * 32), jt = rem >> 5, ln = rem & 31;
    const int jb = 8 * jt + (ln >> 2), b1 = 32 * (ks >> 2) + 8 * (ln & 3) + (ks & 3), b2 = b1 + 4;
    cf v1 = (b1 < B && jb < rb) ? p.Ub[b1 * rb + jb] : make_float2(0.f, 0.f);
    cf v2 = (b2 < B && jb < rb) ? p.Ub[b2 * rb + jb] : make_float2(0.f, 0.f);
    __half r1h, r1l, i1h, i1l, r2h, r2l, i2h, i2l;
    split_f16(v1.x, r1h, r1l); split_f16(v1.y, i1h, i1l);
    split_f16(v2.x, r2h, r2l); split_f16(v2.y, i2h, i2l);
    uint4 hi, lo;
    hi.x = h2_bits(__halves2half2(r1h, i1h)); hi.y = h2_bits(__halves2half2(__hneg(i1h), r1h));
    hi.z = h2_bits(__halves2half2(r2h, i2h)); hi.w = h2_bits(__halves2half2(__hneg(i2h), r2h));
    lo.x = h2_bits(__halves2half2(r1l, i1l)); lo.y = h2_bits(__halves2half2(__hneg(i1l), r1l));
    lo.z = h2_bits(__halves2half2(r2l, i2l)); lo.w = h2_bits(__halves2half2(__hneg(i2l), r2l));
    u1tab[((ks * RBT + jt) * 2 + 0) * 32 + ln] = hi;
    u1tab[((ks * RBT + jt) * 2 + 1) * 32 + ln] = lo;
  }
  for (int idx = tid; idx < A * ldu; idx += nthr) {
    const int a = idx / ldu, j = idx - a * ldu;
    uas[idx] = (j < ra) ? p.Ua[a * ra + j] : make_float2(0.f, 0.f);
  }
  // ---- this thread's first two outputs of a slab: where their partial sums sit ----
  const int n_out = ra * rb;
  int o_src[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int o = tid + i * nthr;
    o_src[i] = -1;
    if (o < n_out) {
      const int ja = o / rb, jb = o - ja * rb;
      o_src[i] = (((ja >> 3) * RBT + (jb >> 3)) * ksplit) * 128 + (4 * (ja & 7) + ((jb & 7) >> 1)) * 4 + (jb & 1);
    }
  }
  if (tid == 0) {
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  const uint32_t nmine = (nslab > blockIdx.x) ? (nslab - blockIdx.x + gstride - 1) / gstride : 0;   // slabs of this block
  if (tid == 0) {
    for (uint32_t i = 0; i < (uint32_t)nbuf && i < nmine; ++i) {
      mbar_expect_tx(&bars[i], G.slab_bytes);
      bulk_g2s(smem + (size_t)i * G.buf_stride, gb + (size_t)(blockIdx.x + i * gstride) * G.slab_bytes, G.slab_bytes, &bars[i]);
    }
  }
  // ---- sparse side: entry bounds three slabs ahead, first entries two slabs ahead ----
  const bool sparse = p.k > 0;
  auto bounds = [&](uint32_t s, int& x0, int& x1) {
    x0 = 0; x1 = 0;
    if (s < nslab) { x0 = (int)p.slab_ptr[s]; x1 = (int)p.slab_ptr[s + 1]; }
  };
  int b0 = 0, b1 = 0, c0 = 0, c1 = 0;
  uint32_t pom = 0, pomc = 0;
  if (sparse) {
    bounds(blockIdx.x, b0, b1);
    bounds(blockIdx.x + gstride, c0, c1);
    if (b0 + tid < b1) pom = p.omega[b0 + tid];
    if (c0 + tid < c1) pomc = p.omega[c0 + tid];
  }

  uint32_t phase = 0;
  int buf = 0, pbuf = 0;
  for (uint32_t it = 0; it < nmine + 2; ++it) {
    const uint32_t s = blockIdx.x + it * gstride;          // slab of stage 1 (valid while it < nmine)
    bool ok = true;
    if (it < nmine) {
      int n0 = 0, n1 = 0;
      if (sparse) bounds(s + 2 * gstride, n0, n1);
      ok = mbar_wait_bounded(&bars[buf], phase);
      uint32_t* xs = reinterpret_cast<uint32_t*>(smem + (size_t)buf * G.buf_stride);
      if (sparse && ok) {
        const uint32_t base = s * E;
        for (int j = b0 + tid, first = 1; j < b1; j += nthr, first = 0) {
          const uint32_t loc = (first ? pom : p.omega[j]) - base;
          const uint32_t xv = xs[loc];
          p.g_s[j] = __half22float2(*reinterpret_cast<const __half2*>(&xv));
          if (!p.keep) xs[loc] = 0u;
        }
        if (b0 + tid < b1) fence_async_smem();   // the zeroed words were written through the generic proxy; a bulk copy overwrites them later
        b0 = c0; b1 = c1; pom = pomc;
        c0 = n0; c1 = n1;
        if (c0 + tid < c1) pomc = p.omega[c0 + tid];
      }
    }
    if (__syncthreads_or(!ok)) {
      if (tid == 0) {
        atomicOr(P.flags, 4);
        uint32_t ph = phase; int bx = buf;
        for (int i = 1; i + 1 < nbuf && it + i < nmine; ++i) {
          if (++bx == nbuf) { bx = 0; ph ^= 1; }
          mbar_wait_bounded(&bars[bx], ph, 1u << 16);
        }
      }
      return;
    }
    // every warp is past its reads of the previous slab: its ring buffer takes the slab nbuf ahead of it
    if (tid == 0 && it >= 1 && it - 1 + nbuf < nmine) {
      mbar_expect_tx(&bars[pbuf], G.slab_bytes);
      bulk_g2s(smem + (size_t)pbuf * G.buf_stride, gb + (size_t)(blockIdx.x + (it - 1 + nbuf) * gstride) * G.slab_bytes,
               G.slab_bytes, &bars[pbuf]);
    }
    // ---- final sum of slab it-2 (its partial tiles were written during iteration it-1) ----
    if (it >= 2) {
      const float* pp = part + (size_t)((it - 1) & 1) * units * 128;
      float* tg_ = reinterpret_cast<float*>(p.t + (size_t)(blockIdx.x + (it - 2) * gstride) * n_out);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (o_src[i] < 0) continue;
        float re = 0.f, im = 0.f;
        for (int kh = 0; kh < ksplit; ++kh) { re += pp[o_src[i] + kh * 128]; im += pp[o_src[i] + kh * 128 + 2]; }
        reinterpret_cast<float2*>(tg_)[tid + i * nthr] = make_float2(re, im);
      }
      for (int o = tid + 2 * nthr; o < n_out; o += nthr) {
        const int ja = o / rb, jb = o - ja * rb;
        const int src = (((ja >> 3) * RBT + (jb >> 3)) * ksplit) * 128 + (4 * (ja & 7) + ((jb & 7) >> 1)) * 4 + (jb & 1);
        float re = 0.f, im = 0.f;
        for (int kh = 0; kh < ksplit; ++kh) { re += pp[src + kh * 128]; im += pp[src + kh * 128 + 2]; }
        reinterpret_cast<float2*>(tg_)[o] = make_float2(re, im);
      }
    }
    // ---- stage 1 of slab it ----
    if (it < nmine) {
      const uint32_t* xs = reinterpret_cast<const uint32_t*>(smem + (size_t)buf * G.buf_stride);
      const uint32_t* xrow = xs + (size_t)(8 * warp + gq) * B;
      float d[RBT][4], dlo[RBT][4];        // the hi and lo parts of Ub accumulate apart: two short chains instead of one
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
        for (int i = 0; i < 4; ++i) { d[jt][i] = 0.f; dlo[jt][i] = 0.f; }
      for (int ks = 0; ks < ks16; ++ks) {
        const int c1_ = 32 * (ks >> 2) + 8 * t + (ks & 3), c2_ = c1_ + 4;
        const uint32_t x1 = c1_ < B ? xrow[c1_] : 0u, x2 = c2_ < B ? xrow[c2_] : 0u;
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          const uint4 h = u1tab[((ks * RBT + jt) * 2 + 0) * 32 + lane], l = u1tab[((ks * RBT + jt) * 2 + 1) * 32 + lane];
          mma_f16(d[jt], h.x, h.y, h.z, h.w, x1, x2);
          mma_f16(dlo[jt], l.x, l.y, l.z, l.w, x1, x2);
        }
      }
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt)
#pragma unroll
        for (int i = 0; i < 4; ++i) d[jt][i] += dlo[jt][i];
      // d0 = Yre[a][jb], d1 = Yre[a+1][jb], d2 = Yim[a][jb], d3 = Yim[a+1][jb], a = 8 warp + 2t, jb = 8 jt + gq
      cf* ys = ysb + (size_t)(it & 1) * A * ldy;
#pragma unroll
      for (int jt = 0; jt < RBT; ++jt) {
        ys[(8 * warp + 2 * t) * ldy + 8 * jt + gq] = make_float2(d[jt][0], d[jt][2]);
        ys[(8 * warp + 2 * t + 1) * ldy + 8 * jt + gq] = make_float2(d[jt][1], d[jt][3]);
      }
    }
    // ---- stage 2 of slab it-1 ----
    if (it >= 1 && it <= nmine) {
      const cf* ys = ysb + (size_t)((it - 1) & 1) * A * ldy;
      float* pw = part + (size_t)(it & 1) * units * 128;
      const int steps = (A / 4) / ksplit;
      for (int unit = warp; unit < units; unit += nwarps) {
        const int tile = unit / ksplit, kh = unit - tile * ksplit, mt = tile / RBT, nt = tile - mt * RBT;
        float tot[4] = {0.f, 0.f, 0.f, 0.f}, acc[4] = {0.f, 0.f, 0.f, 0.f}, acl[4] = {0.f, 0.f, 0.f, 0.f}, acx[4] = {0.f, 0.f, 0.f, 0.f};
        for (int q = 0; q < steps; ++q) {
          const int a = 4 * (kh * steps + q) + t;
          const cf y = ys[a * ldy + 8 * nt + gq], u = uas[a * ldu + 8 * mt + gq];
          float yh0, yl0, yh1, yl1, urh, url, uih, uil;
          split_tf32(y.x, yh0, yl0); split_tf32(y.y, yh1, yl1);
          split_tf32(u.x, urh, url); split_tf32(u.y, uih, uil);
          // rows (re, ja): (ur | ui); rows (im, ja): (-ui | ur)
          // the three products keep their own accumulators: three independent chains
          mma_tf32(acc, urh, -uih, uih, urh, yh0, yh1);
          mma_tf32(acl, url, -uil, uil, url, yh0, yh1);
          mma_tf32(acx, urh, -uih, uih, urh, yl0, yl1);
          if ((q & 15) == 15) {    // the tensor core's accumulator adds truncate: keep its chains short
#pragma unroll
            for (int i = 0; i < 4; ++i) { tot[i] += acc[i] + (acl[i] + acx[i]); acc[i] = 0.f; acl[i] = 0.f; acx[i] = 0.f; }
          }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) tot[i] += acc[i] + (acl[i] + acx[i]);
        *reinterpret_cast<float4*>(pw + (size_t)unit * 128 + lane * 4) = make_float4(tot[0], tot[1], tot[2], tot[3]);
      }
    }
    if (it < nmine) {
      pbuf = buf;
      if (++buf == nbuf) { buf = 0; phase ^= 1; }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Reconstruction of the two trailing modes (half storage), fused with the weight update and the sparse add.
// Two warps share a tile of 16 rows of the slab: each computes the first product for one of the two jb tiles and
// hands its fragments to the other, and each takes half of the column tiles of the second product.  Both products
// run as fp16 m16n8k16 MMAs on two-term fp16 splits of both operands (x = hi + lo / 2048; hi hi, lo hi, hi lo: 22
// bits, the accuracy of the split-TF32 products at half the instructions): the operands here are the factor
// matrices (|u| <= 1) and the expansion of the Adam-normalised core, both far inside the fp16 range.  The slab
// stays fp16 in shared memory: the dense update is rounded to fp16 when it is written back there, the
// sparse term is then added by one thread per entry and rounded again (the storage type is rounded to once after the dense update and once more at Omega),
// and one bulk copy stores the slab.
// ---------------------------------------------------------------------------------------------
struct TailHBGeom {
  int nwarps, nbuf, nbt, ks2;
  uint32_t slab_bytes, buf_stride;
  uint32_t off_ub, off_ua, off_ex, off_bar, total;
};
__host__ inline bool tail_hb_geom(int A, int B, int ra, int rb, TailHBGeom& g) {
  if (A % 16 || A < 16 || A > 128) return false;
  const int rat = (ra + 7) / 8, rbt = (rb + 7) / 8;
  if (rat > 4 || rbt > 2) return false;
  g.nwarps = 2 * (A / 16);
  g.nbt = tc_ksteps(B);
  g.ks2 = 2 * rat;
  g.slab_bytes = (uint32_t)A * B * 4;
  if (g.slab_bytes % 16) return false;
  g.buf_stride = (g.slab_bytes + 127) & ~127u;
  // operand tables in fp16 MMA register order (hi and lo parts), and the exchange buffer of the warp pairs
  const uint32_t ub = (uint32_t)g.nbt * rbt * 32 * 16, ua = (uint32_t)(A / 16) * rat * 2 * 32 * 16;
  const uint32_t ex = (uint32_t)g.nwarps * 32 * 32;
  g.nbuf = 3;
  g.off_ub = 3 * g.buf_stride;
  g.off_ua = g.off_ub + ub;
  g.off_ex = g.off_ua + ua;
  g.off_bar = g.off_ex + ex;
  g.total = g.off_bar + 256;
  return g.total <= 227u * 1024u;
}
struct TailHBParams {
  TailParams p;
  TailHBGeom g;
  int* flags;
};

// NBT > 0 (odd): the number of column tiles is built in, which fixes B = 4 (NBT - 1) + 1; a warp's share of the tile
// loop is unrolled and every offset into a row is an immediate.  NBT = 0: both at run time.
template <int RAT, int RBT, int NBT>
__global__ void __launch_bounds__(512, 1) back_tail_h_kernel(void* __restrict__ w, TailHBParams P) {
  griddep_chain();
  extern __shared__ __align__(128) unsigned char smem[];
  const TailParams& p = P.p;
  const TailHBGeom& G = P.g;
  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  const int A = p.A, B = NBT ? 4 * (NBT - 1) + 1 : p.B, ra = p.ra, rb = p.rb, nbuf = G.nbuf, nbt = NBT ? NBT : G.nbt;
  constexpr int KS2 = 2 * RAT;
  const uint32_t E = p.E, nslab = p.nslab, gstride = gridDim.x;
  const int mtile = warp >> 1, am = 16 * mtile, r0 = am + gq, r1 = r0 + 8;
  const int nbh = (nbt + 1) / 2, nb0 = (warp & 1) ? nbh : 0, nb1 = (warp & 1) ? nbt : nbh;   // this warp's column tiles
  uint4* ubf = reinterpret_cast<uint4*>(smem + G.off_ub);       // [nbt][RBT][32]: fp16 pairs (b0.hi, b1.hi, b0.lo, b1.lo)
  uint4* uaf = reinterpret_cast<uint4*>(smem + G.off_ua);       // [A/16][RAT][hi|lo][32]
  uint4* exch = reinterpret_cast<uint4*>(smem + G.off_ex);      // [warps][32][2]: Y' fragments handed to the partner warp
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G.off_bar);
  unsigned char* wb = static_cast<unsigned char*>(w);

  // Ub as stage-2 operand fragments of the fp16 m16n8k16 shape, per column tile, jb tile and lane (g, t):
  //   n = g <-> (b, c), b = 16 (nb>>2) + (nb&3) + 4 (g>>1), c = g & 1;  k = 2t, 2t+1 <-> (jb, re), (jb+1, re),
  //   k = 2t+8, 2t+9 <-> (jb, im), (jb+1, im), jb = 8 jt + 2t;
  //   W3[(jb,re)][(b,re)] = ur, [(b,im)] = ui;  W3[(jb,im)][(b,re)] = -ui, [(b,im)] = ur.
  // Each value as hi + lo / 2048 with hi and lo in fp16 (22 bits together; |u| <= 1).
  for (int idx = tid; idx < nbt * RBT * 32; idx += nthr) {
    const int nb = idx / (RBT * 32), rem = idx - nb * (RBT * 32), jt = rem >> 5, ln = rem & 31, g_ = ln >> 2, t_ = ln & 3;
    const int bq = 16 * (nb >> 2) + (nb & 3) + 4 * (g_ >> 1), jb = 8 * jt + 2 * t_;
    const bool odd = g_ & 1;
    const cf va = (bq < B && jb < rb) ? p.Ub[bq * rb + jb] : make_float2(0.f, 0.f);
    const cf vb = (bq < B && jb + 1 < rb) ? p.Ub[bq * rb + jb + 1] : make_float2(0.f, 0.f);
    const float re0 = odd ? va.y : va.x, re1 = odd ? vb.y : vb.x;         // rows (jb, re), (jb+1, re) of column n
    const float im0 = odd ? va.x : -va.y, im1 = odd ? vb.x : -vb.y;       // rows (jb, im), (jb+1, im)
    __half h[4], l[4];
    split_f16_scaled(re0, h[0], l[0]); split_f16_scaled(re1, h[1], l[1]);
    split_f16_scaled(im0, h[2], l[2]); split_f16_scaled(im1, h[3], l[3]);
    ubf[idx] = make_uint4(h2_bits(__halves2half2(h[0], h[1])), h2_bits(__halves2half2(h[2], h[3])),
                          h2_bits(__halves2half2(l[0], l[1])), h2_bits(__halves2half2(l[2], l[3])));
  }
  // Ua as stage-1 operand fragments of the fp16 m16n8k16 shape, per row tile, step ks and lane (g, t): rows
  // q0 = 16 mt + g and q0 + 8; k = 2t, 2t+1 <-> (ja, re), (ja+1, re), k = 2t+8, 2t+9 <-> (ja, im), (ja+1, im),
  // ja = 8 ks + 2t:  a0 = re(q0), a1 = re(q0+8), a2 = im(q0), a3 = im(q0+8), each a pair over (ja, ja+1); hi, then lo
  for (int idx = tid; idx < (A / 16) * RAT * 32; idx += nthr) {
    const int mt = idx / (RAT * 32), rem = idx - mt * (RAT * 32), ks = rem >> 5, ln = rem & 31;
    const int ja = 8 * ks + 2 * (ln & 3), q0 = 16 * mt + (ln >> 2), q1 = q0 + 8;
    const cf z = make_float2(0.f, 0.f);
    const cf u00 = (ja < ra) ? p.Ua[q0 * ra + ja] : z, u01 = (ja + 1 < ra) ? p.Ua[q0 * ra + ja + 1] : z;
    const cf u10 = (ja < ra) ? p.Ua[q1 * ra + ja] : z, u11 = (ja + 1 < ra) ? p.Ua[q1 * ra + ja + 1] : z;
    const float v[8] = {u00.x, u01.x, u10.x, u11.x, u00.y, u01.y, u10.y, u11.y};
    __half h[8], l[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) split_f16_scaled(v[e], h[e], l[e]);
    uaf[((mt * RAT + ks) * 2 + 0) * 32 + ln] = make_uint4(h2_bits(__halves2half2(h[0], h[1])), h2_bits(__halves2half2(h[2], h[3])),
                                                          h2_bits(__halves2half2(h[4], h[5])), h2_bits(__halves2half2(h[6], h[7])));
    uaf[((mt * RAT + ks) * 2 + 1) * 32 + ln] = make_uint4(h2_bits(__halves2half2(l[0], l[1])), h2_bits(__halves2half2(l[2], l[3])),
                                                          h2_bits(__halves2half2(l[4], l[5])), h2_bits(__halves2half2(l[6], l[7])));
  }
  if (tid == 0) {
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  const uint32_t nmine = (nslab > blockIdx.x) ? (nslab - blockIdx.x + gstride - 1) / gstride : 0;
  if (tid == 0 && nmine > 0) {
    mbar_expect_tx(&bars[0], G.slab_bytes);
    bulk_g2s(smem, wb + (size_t)blockIdx.x * G.slab_bytes, G.slab_bytes, &bars[0]);
  }
  const bool sparse = p.k > 0;
  auto bounds = [&](uint32_t s, int& x0, int& x1) {
    x0 = 0; x1 = 0;
    if (s < nslab) { x0 = (int)p.slab_ptr[s]; x1 = (int)p.slab_ptr[s + 1]; }
  };
  int b0 = 0, b1 = 0, n0 = 0, n1 = 0;
  uint32_t pom = 0; cf pn = make_float2(0.f, 0.f);
  if (sparse) {
    bounds(blockIdx.x, b0, b1);
    bounds(blockIdx.x + gstride, n0, n1);
    if (b0 + tid < b1) { pom = p.omega[b0 + tid]; pn = p.n_s[b0 + tid]; }
  }
  const bool decay = p.decay != 1.0f;
  uint32_t phase = 0;
  int buf = 0, lbuf = 1;            // ring slot of this iteration and of the slab loaded one ahead
  for (uint32_t it = 0; it < nmine; ++it) {
    const uint32_t s = blockIdx.x + it * gstride;
    if (tid == 0) bulk_wait_read<1>();          // the store of two iterations ago has read its buffer
    // T' fragments for stage 1 (in flight while the slab arrives): T'[ja = 8 ks + 2t + e][jb = 8 jt + gq], e = 0, 1,
    // for the jb tiles this warp computes: with two jb tiles the two warps of a row tile take one each
    constexpr int NJ = (RBT == 2) ? 1 : RBT;          // jb tiles whose stage 1 this warp computes
    const int jt0 = (RBT == 2) ? (warp & 1) : 0;
    cf tv[RAT][NJ][2];
    {
      const cf* tin = p.t + (size_t)s * ra * rb;
#pragma unroll
      for (int ks = 0; ks < RAT; ++ks)
#pragma unroll
        for (int j = 0; j < NJ; ++j)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int ja = 8 * ks + 2 * t + e, jb = 8 * (jt0 + j) + gq;
            tv[ks][j][e] = (ja < ra && jb < rb) ? __ldg(tin + (size_t)ja * rb + jb) : make_float2(0.f, 0.f);
          }
    }
    const bool ok = mbar_wait_bounded(&bars[buf], phase);
    if (__syncthreads_or(!ok)) {
      if (tid == 0) { atomicOr(P.flags, 4); bulk_wait_all<0>(); }
      return;
    }
    if (tid == 0 && it + 1 < nmine) {             // buffer lbuf was stored two iterations ago (read checked above)
      mbar_expect_tx(&bars[lbuf], G.slab_bytes);
      bulk_g2s(smem + (size_t)lbuf * G.buf_stride, wb + (size_t)(s + gstride) * G.slab_bytes, G.slab_bytes, &bars[lbuf]);
    }
    uint32_t* ws = reinterpret_cast<uint32_t*>(smem + (size_t)buf * G.buf_stride);     // half2 words [A][B]
    {
      // ---- stage 1: Y'[a][(c, jb)] for rows r0 and r1, fp16 m16n8k16 on two-term splits of both operands
      //      (re tile: B = (Tr | -Ti), im tile: B = (Ti | Tr); hi hi into one accumulator, lo hi and hi lo, which
      //      carry the factor 2048, into another) ----
      float d1[2][NJ][4];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        float eh[2][4], el[2][4];
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 4; ++i) { eh[c][i] = 0.f; el[c][i] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < RAT; ++ks) {
          const uint4 uh = uaf[((mtile * RAT + ks) * 2 + 0) * 32 + lane], ul = uaf[((mtile * RAT + ks) * 2 + 1) * 32 + lane];
          const cf t0 = tv[ks][j][0], t1 = tv[ks][j][1];
          const __half2 rh = __floats2half2_rn(t0.x, t1.x), ih = __floats2half2_rn(t0.y, t1.y);
          const float2 rb_ = __half22float2(rh), ib_ = __half22float2(ih);
          const __half2 rl = __floats2half2_rn((t0.x - rb_.x) * kF16LoScale, (t1.x - rb_.y) * kF16LoScale);
          const __half2 il = __floats2half2_rn((t0.y - ib_.x) * kF16LoScale, (t1.y - ib_.y) * kF16LoScale);
          const uint32_t trh = h2_bits(rh), tih = h2_bits(ih), trl = h2_bits(rl), til = h2_bits(il);
          const uint32_t nih = tih ^ 0x80008000u, nil = til ^ 0x80008000u;        // -Ti
          mma_f16(eh[0], uh.x, uh.y, uh.z, uh.w, trh, nih);
          mma_f16(el[0], ul.x, ul.y, ul.z, ul.w, trh, nih);
          mma_f16(el[0], uh.x, uh.y, uh.z, uh.w, trl, nil);
          mma_f16(eh[1], uh.x, uh.y, uh.z, uh.w, tih, trh);
          mma_f16(el[1], ul.x, ul.y, ul.z, ul.w, tih, trh);
          mma_f16(el[1], uh.x, uh.y, uh.z, uh.w, til, trl);
        }
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 4; ++i) d1[c][j][i] = eh[c][i] + el[c][i] * kF16LoInv;
      }
      // Y' as fp16 m16n8k16 A fragments, hi and lo (scaled by 2048): a0 = (row g; jb, jb+1; re), a1 = (row g+8; re),
      // a2 = (row g; im), a3 = (row g+8; im) -- the accumulator pairs of stage 1 as they are.  Y' is built from the
      // Adam-normalised core through factors with orthonormal columns, so its entries are far inside the fp16 range.
      uint32_t ymh[NJ][4], yml[NJ][4];                 // of the jb tiles this warp computed
#pragma unroll
      for (int j = 0; j < NJ; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int hrow = 0; hrow < 2; ++hrow) {
            const float v0 = d1[c][j][2 * hrow], v1 = d1[c][j][2 * hrow + 1];
            const __half2 hh = __floats2half2_rn(v0, v1);
            const float2 back = __half22float2(hh);
            ymh[j][2 * c + hrow] = h2_bits(hh);
            yml[j][2 * c + hrow] = h2_bits(__floats2half2_rn((v0 - back.x) * kF16LoScale, (v1 - back.y) * kF16LoScale));
          }
      uint32_t yh[RBT][4], yl[RBT][4];
      if (RBT == 2) {
        // hand this warp's jb tile to the partner warp of the row tile and take the partner's (one named barrier per
        // pair of warps; the block barrier further down keeps the next iteration's writes behind these reads)
        exch[(warp * 32 + lane) * 2 + 0] = make_uint4(ymh[0][0], ymh[0][1], ymh[0][2], ymh[0][3]);
        exch[(warp * 32 + lane) * 2 + 1] = make_uint4(yml[0][0], yml[0][1], yml[0][2], yml[0][3]);
        asm volatile("barrier.sync %0, 64;" ::"r"(1 + mtile) : "memory");
        const uint4 oh = exch[((warp ^ 1) * 32 + lane) * 2 + 0], ol = exch[((warp ^ 1) * 32 + lane) * 2 + 1];
        const uint32_t oth[4] = {oh.x, oh.y, oh.z, oh.w}, otl[4] = {ol.x, ol.y, ol.z, ol.w};
        const bool second = (warp & 1) != 0;           // this warp computed jb tile 1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          yh[0][i] = second ? oth[i] : ymh[0][i]; yh[RBT - 1][i] = second ? ymh[0][i] : oth[i];
          yl[0][i] = second ? otl[i] : yml[0][i]; yl[RBT - 1][i] = second ? yml[0][i] : otl[i];
        }
      } else {
#pragma unroll
        for (int j = 0; j < NJ; ++j)
#pragma unroll
          for (int i = 0; i < 4; ++i) { yh[j][i] = ymh[j][i]; yl[j][i] = yml[j][i]; }
      }
      // ---- stage 2, one column tile at a time, applied to the slab right away: three fp16 products per jb tile
      //      (hi hi, lo hi, hi lo), the two small ones summed and scaled back by 1/2048 ----
      constexpr int NB_UNROLL = NBT ? (NBT + 1) / 2 : 1;
#pragma unroll NB_UNROLL
      for (int nb = nb0; nb < nb1; ++nb) {
        float dh[4] = {0.f, 0.f, 0.f, 0.f}, dl[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int jt = 0; jt < RBT; ++jt) {
          const uint4 f = ubf[(nb * RBT + jt) * 32 + lane];
          mma_f16(dh, yh[jt][0], yh[jt][1], yh[jt][2], yh[jt][3], f.x, f.y);
          mma_f16(dl, yl[jt][0], yl[jt][1], yl[jt][2], yl[jt][3], f.x, f.y);
          mma_f16(dl, yh[jt][0], yh[jt][1], yh[jt][2], yh[jt][3], f.z, f.w);
        }
        float dx[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) { dl[i] *= kF16LoInv; dx[i] = 0.f; }
        // d0 + i d1 = D[r0][b], d2 + i d3 = D[r1][b] with b = 16 (nb>>2) + (nb&3) + 4 t
        const int bo = 16 * (nb >> 2) + (nb & 3) + 4 * t;
        if (bo < B) {
          uint32_t* p0 = ws + (size_t)r0 * B + bo;
          uint32_t* p1 = ws + (size_t)r1 * B + bo;
          const uint32_t w0 = *p0, w1 = *p1;
          float2 v0 = __half22float2(*reinterpret_cast<const __half2*>(&w0));
          float2 v1 = __half22float2(*reinterpret_cast<const __half2*>(&w1));
          if (decay) { v0.x *= p.decay; v0.y *= p.decay; v1.x *= p.decay; v1.y *= p.decay; }
          v0.x = fmaf(-p.s_low, dh[0] + (dl[0] + dx[0]), v0.x); v0.y = fmaf(-p.s_low, dh[1] + (dl[1] + dx[1]), v0.y);
          v1.x = fmaf(-p.s_low, dh[2] + (dl[2] + dx[2]), v1.x); v1.y = fmaf(-p.s_low, dh[3] + (dl[3] + dx[3]), v1.y);
          *p0 = h2_bits(__floats2half2_rn(v0.x, v0.y));
          *p1 = h2_bits(__floats2half2_rn(v1.x, v1.y));
        }
      }
    }
    __syncthreads();                                   // the dense update of the slab is complete (rounded to fp16)
    // ---- scaled sparse add at Omega, one entry per thread, rounded again ----
    if (sparse) {
      const uint32_t base = s * E;
      for (int j = b0 + tid, first = 1; j < b1; j += nthr, first = 0) {
        const uint32_t loc = (first ? pom : p.omega[j]) - base;
        const cf n = first ? pn : p.n_s[j];
        const uint32_t wv = ws[loc];
        float2 v = __half22float2(*reinterpret_cast<const __half2*>(&wv));
        v.x = fmaf(-p.s_sparse, n.x, v.x); v.y = fmaf(-p.s_sparse, n.y, v.y);
        ws[loc] = h2_bits(__floats2half2_rn(v.x, v.y));
      }
      b0 = n0; b1 = n1;
      if (b0 + tid < b1) { pom = p.omega[b0 + tid]; pn = p.n_s[b0 + tid]; }
      bounds(s + 2 * gstride, n0, n1);
    }
    fence_async_smem();                                // order the shared-memory writes before the bulk store reads them
    __syncthreads();
    if (tid == 0) {
      bulk_s2g(wb + (size_t)s * G.slab_bytes, smem + (size_t)buf * G.buf_stride, G.slab_bytes);
      bulk_commit();
    }
    if (++buf == nbuf) { buf = 0; phase ^= 1; }
    if (++lbuf == nbuf) lbuf = 0;
  }
  if (tid == 0) bulk_wait_all<0>();   // stores complete before the block's shared memory goes away
}

}  // namespace tg
