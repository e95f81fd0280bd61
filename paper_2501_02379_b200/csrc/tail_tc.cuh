// Fast path of the two streaming kernels of a step (complex64 storage, trailing slab of
// A x B entries with A in {16, 32, 64}, B <= 33, r_{N-1} <= 16, r_N <= 8).
//
// A thread block works on one group of consecutive slabs at a time.  Groups arrive by bulk
// asynchronous copy into a ring in shared memory that the whole block shares, and a block keeps
// several groups in flight.  The compression kernel runs blocks of four warps, four blocks per SM;
// the reconstruction kernel blocks of eight warps, two per SM (16 warps per SM either way).  The two
// trailing mode products run on the tensor cores as split-precision TF32 (x = hi + lo, the
// three products hi*hi, lo*hi, hi*lo, fp32 accumulation), chained through registers: the
// accumulator fragments of the first product are the operand fragments of the second.  The
// factor-matrix fragments a warp needs never change (a warp always owns the same rows of a
// slab): the reconstruction keeps them in registers for the whole kernel, the compression reads
// them from small tables in shared and global memory laid out in MMA register order.
//
// Complex arithmetic is carried as real arithmetic on interleaved (re, im) data:
//   Y = X conj(Ub):   [Yre; Yim] = W1 [Xre; Xim],  W1 = [[ur, ui], [-ui, ur]]
//   T = conj(Ua)^T Y: [Tre; Tim] = W2 [Yre; Yim],  W2 = [[ur, ui], [-ui, ur]]
// and without conjugation for the reconstruction.  The K index inside one MMA step is a free
// permutation as long as both operands use the same one; it is chosen so that every operand
// load from the slab is one conflict-free 8-byte shared-memory access.
#pragma once
#include "common.cuh"
#include "ptx.cuh"
#include "tail.cuh"

namespace tg {

constexpr int TC_WARPS = 8;
constexpr int TC_THREADS = 32 * TC_WARPS;
constexpr uint32_t TC_SMEM_PER_BLOCK = 113 * 1024;   // two blocks per SM

struct TcGeom {
  int nbuf;                 // ring depth in groups
  int spi;                  // slabs per group
  int tps;                  // row tiles per slab, one warp each (spi * tps == 8)
  int nbt;                  // reconstruction: column tiles of 4 complex entries that hold any b < B
  uint32_t ngroups;
  uint32_t slab_bytes, grp_stride;
  uint32_t off_aux;         // compression: partial-sum scratch; reconstruction: Ub fragment table
  uint32_t off_bar;
  uint32_t total;
};

struct TailTcParams {
  TailParams p;
  TcGeom g;
  int* flags;               // sticky status word (bit 4: a bulk copy did not arrive within the wait limit)
  float s_sparse_pre;       // eta*lambda / (1 - eta*wd): the sparse term is applied before the decayed dense update
  const float4* u2tab;      // compression: stage-2 operand fragments of Ua (proj_u2tab_kernel)
};

// k-steps of the compression's first product that hold any (b, re|im) of a row of 2B floats
__host__ __device__ inline int tc_ksteps(int B) {
  const int twoB = 2 * B, KB = twoB / 32, rem = twoB - 32 * KB;
  return 4 * KB + (rem >= 8 ? 4 : rem / 2);
}

__host__ inline bool tail_tc_geom(bool back, int A, int B, int rat, uint32_t nslab, int ns, TcGeom& g) {
  const int rows = back ? 16 : 8;
  if (A % rows) return false;
  g.tps = A / rows;
  if (g.tps < 1 || g.tps > TC_WARPS || TC_WARPS % g.tps) return false;
  g.spi = (TC_WARPS / g.tps) * ns;     // ns slabs per warp and iteration (small slabs)
  g.nbt = tc_ksteps(B);
  g.slab_bytes = (uint32_t)A * B * 8;
  g.grp_stride = ((uint32_t)g.spi * g.slab_bytes + 127) & ~127u;
  g.ngroups = (nslab + g.spi - 1) / g.spi;
  const uint32_t aux = back ? (uint32_t)g.nbt * 2 * 32 * 16 : 2u * TC_WARPS * rat * 128 * 4;
  const uint32_t fixed = ((aux + 127) & ~127u) + 128;
  if (fixed + 2 * g.grp_stride > TC_SMEM_PER_BLOCK) return false;
  int nbuf = (int)((TC_SMEM_PER_BLOCK - fixed) / g.grp_stride);
  if (nbuf > 8) nbuf = 8;
  if (nbuf < (back ? 3 : 2)) return false;
  g.nbuf = nbuf;
  g.off_aux = (uint32_t)nbuf * g.grp_stride;
  g.off_bar = g.off_aux + ((aux + 127) & ~127u);
  g.total = g.off_bar + 128;
  return true;
}

// x = hi + lo with hi a TF32 value (10 explicit mantissa bits, rounded to nearest by adding half a
// unit in the last kept place to the bit pattern) and lo = x - hi exact in fp32.  Integer ops
// instead of cvt.rna.tf32.f32, which issues on the quarter-rate conversion pipe.
__device__ __forceinline__ void split_tf32(float x, float& hi, float& lo) {
  hi = __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
  lo = x - hi;
}

// The same with hi truncated instead of rounded (one integer op less).  lo = x - hi is still exact; it is
// at most 2^-10 |x| instead of 2^-11 |x|, so what the tensor core drops of it is at most 2^-20 |x|.
__device__ __forceinline__ void split_tf32_trunc(float x, float& hi, float& lo) {
  hi = __uint_as_float(__float_as_uint(x) & 0xffffe000u);
  lo = x - hi;
}

// one group of slabs -> ring buffer `buf`
__device__ __forceinline__ void tc_issue_load(const unsigned char* gbase, unsigned char* smem, const TcGeom& G,
                                              uint64_t* bars, uint32_t u, int buf, uint32_t nslab) {
  uint32_t nv = nslab - u * (uint32_t)G.spi;
  if (nv > (uint32_t)G.spi) nv = (uint32_t)G.spi;
  const uint32_t bytes = nv * G.slab_bytes;
  mbar_expect_tx(&bars[buf], bytes);
  bulk_g2s(smem + (size_t)buf * G.grp_stride, gbase + (size_t)u * G.spi * G.slab_bytes, bytes, &bars[buf]);
}

// ---------------------------------------------------------------------------------------------
// Compression of the two trailing modes, fused with the sparse gather / Adam / residual.
//   stage 1  D1[(c,jb)][a] = sum_{(b,c')} W1[(c,jb)][(b,c')] X[a][(b,c')]     m16 = (re|im) x 8 jb, n8 = 8 rows a (one row tile)
//            step ks: k = t <-> (b, re), k = t+4 <-> (b, im), float offset of b in the row f = 32 (ks>>2) + 8 t + 2 (ks&3)
//   stage 2  D2[(c,ja)][jb] = sum_{(a,c')} W2[(c,ja)][(a,c')] Y[(a,c')][jb]   m16 = (re|im) x 8 ja, n8 = 8 jb
//            step c: k = t <-> (a, c), k = t+4 <-> (a+1, c), a = a0 + 2 t   (the accumulator layout of stage 1)
// A block has PJ_WARPS warps; a warp owns NTW row tiles of one slab of the group (tiles wt, wt + tw, ...,
// tw = warps per slab) and accumulates stage 2 over them.  The warps' partial D2 are summed through
// shared memory, in warp order, one iteration later (so that one block-wide barrier per iteration suffices).
// RAT = ceil(ra/8); KS = k-steps of stage 1 (>= tc_ksteps(B)).
// ---------------------------------------------------------------------------------------------

__host__ inline bool proj_tc_geom(int A, int B, int rat, uint32_t nslab, int ntw, int PJ_WARPS, uint32_t smem_per_block, TcGeom& g) {   // PJ_WARPS: warps per block
  if (A % 8) return false;
  const int tiles = A / 8;
  // tps = warps per slab, each with ntw row tiles; spi = slabs per group
  if (tiles % ntw) return false;
  g.tps = tiles / ntw;
  if (g.tps > PJ_WARPS || PJ_WARPS % g.tps) return false;
  g.spi = PJ_WARPS / g.tps;
  g.nbt = tc_ksteps(B);
  g.slab_bytes = (uint32_t)A * B * 8;
  g.grp_stride = ((uint32_t)g.spi * g.slab_bytes + 127) & ~127u;
  g.ngroups = (nslab + g.spi - 1) / g.spi;
  const uint32_t aux = 2u * PJ_WARPS * rat * 128 * 4 + (uint32_t)g.nbt * 32 * 32;   // partial sums, then the Ub fragment table
  const uint32_t fixed = ((aux + 127) & ~127u) + 128;
  if (fixed + 2 * g.grp_stride > smem_per_block) return false;
  int nbuf = (int)((smem_per_block - fixed) / g.grp_stride);
  if (nbuf > 8) nbuf = 8;
  g.nbuf = nbuf;
  g.off_aux = (uint32_t)nbuf * g.grp_stride;
  g.off_bar = g.off_aux + ((aux + 127) & ~127u);
  g.total = g.off_bar + 128;
  return true;
}

// Stage-2 operand fragments of the compression kernel: for row tile `tile`, ja tile `mt` and lane (gq, t), with
// a = 8 tile + 2 t and ja = 8 mt + gq: (u0.hi.x, u0.hi.y, u1.hi.x, u1.hi.y), (u0.lo.x, u0.lo.y, u1.lo.x, u1.lo.y),
// u0 = Ua[a][ja], u1 = Ua[a+1][ja] split as TF32 value + remainder.  Rebuilt whenever Ua changes.
__global__ void proj_u2tab_kernel(const cf* __restrict__ Ua, int A, int ra, int rat, float4* __restrict__ tab) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (A / 8) * rat * 32) return;
  const int ln = idx & 31, mt = (idx >> 5) % rat, tile = (idx >> 5) / rat, g_ = ln >> 2, t_ = ln & 3;
  const int a = 8 * tile + 2 * t_, ja = 8 * mt + g_;
  const cf v0 = (ja < ra) ? Ua[a * ra + ja] : make_float2(0.f, 0.f);
  const cf v1 = (ja < ra) ? Ua[(a + 1) * ra + ja] : make_float2(0.f, 0.f);
  cf h0, l0, h1, l1;
  split_tf32(v0.x, h0.x, l0.x); split_tf32(v0.y, h0.y, l0.y);
  split_tf32(v1.x, h1.x, l1.x); split_tf32(v1.y, h1.y, l1.y);
  tab[2 * idx] = make_float4(h0.x, h0.y, h1.x, h1.y);
  tab[2 * idx + 1] = make_float4(l0.x, l0.y, l1.x, l1.y);
}

constexpr int PJ_WARPS = 4;

// TW = warps per slab (row tiles of a slab / NTW): 4, 2 or 1, so a group has PJ_WARPS / TW slabs
template <int RAT, int KS, int NTW, int TW>
__global__ void __launch_bounds__(32 * PJ_WARPS, 4) proj_tail_tc_kernel(const void* __restrict__ g, TailTcParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  constexpr int PJ_THREADS = 32 * PJ_WARPS;
  const TailParams& p = P.p;
  const TcGeom& G = P.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  constexpr int tw = TW, spi = PJ_WARPS / TW;
  // an odd KS fixes B = 4 (KS - 1) + 1 and NTW * TW fixes the rows of a slab, so that every offset into a slab
  // is an immediate
  const int B = (KS & 1) ? 4 * (KS - 1) + 1 : p.B;
  const int ra = p.ra, rb = p.rb, twoB = 2 * B, nbuf = G.nbuf;
  const uint32_t E = (KS & 1) ? (uint32_t)(8 * NTW * TW * (4 * (KS - 1) + 1)) : p.E;
  const uint32_t nslab = p.nslab, ngroups = G.ngroups, gstride = gridDim.x;
  const int q = warp / tw, wt = warp - q * tw;
  constexpr int REDW = RAT * 128;                       // floats of one warp's partial: [8 RAT][8] complex
  float* red = reinterpret_cast<float*>(smem + G.off_aux);   // [2][PJ_WARPS][REDW]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G.off_bar);
  const unsigned char* gb = static_cast<const unsigned char*>(g);

  // ---- Ub as stage-1 operand fragments, per k-step and lane, in MMA register order (a0, a1, a2, a3) =
  //      (ur, -ui, ui, ur) of Ub[b][jb = gq]: [0] of the TF32 part, [1] of the remainder ----
  float4* u1tab = reinterpret_cast<float4*>(red + 2 * PJ_WARPS * REDW);   // [2][nbt][32]
  for (int idx = tid; idx < G.nbt * 32; idx += PJ_THREADS) {
    const int ks = idx >> 5, ln = idx & 31, g_ = ln >> 2, t_ = ln & 3;
    const int f = 32 * (ks >> 2) + 8 * t_ + 2 * (ks & 3);
    cf u = (f < twoB && g_ < rb) ? p.Ub[(f >> 1) * rb + g_] : make_float2(0.f, 0.f);
    cf h, l; split_tf32(u.x, h.x, l.x); split_tf32(u.y, h.y, l.y);
    u1tab[idx] = make_float4(h.x, -h.y, h.y, h.x);
    u1tab[G.nbt * 32 + idx] = make_float4(l.x, -l.y, l.y, l.x);
  }
  // ---- stage-2 operand fragments come from the table in global memory (L1-resident): two float4 per
  //      (row tile, ja tile, lane), read again for every slab so that they hold no registers across the loop ----
  const float4* u2p[NTW];
#pragma unroll
  for (int nt = 0; nt < NTW; ++nt) u2p[nt] = P.u2tab + ((size_t)(wt + nt * tw) * RAT * 32 + lane) * 2;
  // ---- this thread's first two output floats of a group: which partial element each sums, where it goes ----
  const int out_per_slab = 2 * ra * rb, n_out = spi * out_per_slab;
  int o_src[2], o_dst[2], o_q[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int o = tid + i * PJ_THREADS;
    o_src[i] = -1; o_dst[i] = 0; o_q[i] = 0;
    if (o < n_out) {
      const int qo = o / out_per_slab, rem = o - qo * out_per_slab;
      const int cidx = rem >> 1, ja = cidx / rb, jb = cidx - ja * rb;
      o_src[i] = qo * tw * REDW + (ja * 8 + jb) * 2 + (rem & 1);
      o_dst[i] = qo * out_per_slab + rem; o_q[i] = qo;
    }
  }

  // the last column's factor row for the FMA path of an odd KS: Ub[B-1][gq]
  const cf ulast = ((KS & 1) && gq < rb) ? p.Ub[(size_t)(B - 1) * rb + gq] : make_float2(0.f, 0.f);
  if (tid == 0) {
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  griddep_chain();            // so far only Ub was read: the tables are built while the previous kernel drains
  if (tid == 0) {
    uint32_t u = blockIdx.x;
    for (int i = 0; i < nbuf && u < ngroups; ++i, u += gstride) tc_issue_load(gb, smem, G, bars, u, i, nslab);
  }
  // ---- sparse side, software-pipelined: a group's entry bounds are fetched three groups ahead, its first
  //      entries (one per thread) two groups ahead, so that neither load is waited for ----
  const bool sparse = p.k > 0;
  auto bounds = [&](uint32_t ug, int& x0, int& x1) {
    x0 = 0; x1 = 0;
    if (ug < ngroups) {
      uint32_t e = (ug + 1) * spi; if (e > nslab) e = nslab;
      x0 = (int)p.slab_ptr[ug * spi]; x1 = (int)p.slab_ptr[e];
    }
  };
  int b0 = 0, b1 = 0, c0 = 0, c1 = 0;
  uint32_t pom = 0, pomc = 0;
  if (sparse) {
    bounds(blockIdx.x, b0, b1);
    bounds(blockIdx.x + gstride, c0, c1);
    if (b0 + tid < b1) pom = p.omega[b0 + tid];
    if (c0 + tid < c1) pomc = p.omega[c0 + tid];
  }

  // sums the partials of iteration `itp` (group up) in warp order and writes T
  auto reduce_out = [&](uint32_t up, uint32_t itp) {
    const float* rp = red + (size_t)(itp & 1) * PJ_WARPS * REDW;
    float* tg_ = reinterpret_cast<float*>(p.t) + (size_t)up * spi * out_per_slab;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      if (o_src[i] >= 0 && up * spi + o_q[i] < nslab) {
        const float* src = rp + o_src[i];
        float acc = src[0];
#pragma unroll
        for (int w = 1; w < tw; ++w) acc += src[(size_t)w * REDW];
        tg_[o_dst[i]] = acc;
      }
    }
    for (int o = tid + 2 * PJ_THREADS; o < n_out; o += PJ_THREADS) {     // wide cores: more outputs than 2 per thread
      const int qo = o / out_per_slab, rem = o - qo * out_per_slab;
      const int cidx = rem >> 1, ja = cidx / rb, jb = cidx - ja * rb;
      if (up * spi + qo >= nslab) continue;
      const float* src = rp + (size_t)(qo * tw) * REDW + ((ja * 8 + jb) * 2 + (rem & 1));
      float acc = src[0];
      for (int w = 1; w < tw; ++w) acc += src[(size_t)w * REDW];
      tg_[o] = acc;
    }
  };

  uint32_t it = 0, phase = 0;
  int buf = 0, pbuf = 0;      // ring slot of this iteration and of the previous one
  for (uint32_t u = blockIdx.x; u < ngroups; u += gstride, ++it) {
    // entry bounds of the group after next: issued now, used at the end of this iteration
    int n0 = 0, n1 = 0;
    if (sparse) bounds(u + 2 * gstride, n0, n1);
    const bool ok = mbar_wait_bounded(&bars[buf], phase);
    float* xg = reinterpret_cast<float*>(smem + (size_t)buf * G.grp_stride);
    // ---- sparse part, before the barrier: gather and zero (the residual); one entry of the group per thread ----
    const int jcur = b0 + tid;
    if (sparse && ok) {
      // the gathered values go to the sparse-value buffer; their Adam update runs with the core's
      const uint32_t base = u * (uint32_t)spi * E;
      if (jcur < b1) {
        cf* xp = reinterpret_cast<cf*>(xg) + (pom - base);
        p.g_s[jcur] = *xp;
        if (!p.keep) *xp = make_float2(0.f, 0.f);
      }
      for (int j = jcur + PJ_THREADS; j < b1; j += PJ_THREADS) {   // more entries than threads: not prefetched
        cf* xp = reinterpret_cast<cf*>(xg) + (p.omega[j] - base);
        p.g_s[j] = *xp;
        if (!p.keep) *xp = make_float2(0.f, 0.f);
      }
    }
    if (__syncthreads_or(!ok)) {
      // a copy did not arrive: record it, let the copies still in flight land (bounded), leave
      if (tid == 0) {
        atomicOr(P.flags, 4);
        uint32_t ux = u + gstride, ph = phase;
        int bx = buf;
        for (int i = 1; i + 1 < nbuf && ux < ngroups; ++i, ux += gstride) {
          if (++bx == nbuf) { bx = 0; ph ^= 1; }
          mbar_wait_bounded(&bars[bx], ph, 1u << 16);
        }
      }
      return;
    }
    // every warp is past its reads of the previous group: its ring buffer takes the group nbuf ahead
    if (it > 0 && tid == 0) {
      const uint32_t un = u + (uint32_t)(nbuf - 1) * gstride;
      if (un < ngroups) tc_issue_load(gb, smem, G, bars, un, pbuf, nslab);
    }
    // ---- this group's contraction ----
    float d2[RAT][2][4];
    if (u * spi + q < nslab) {
      // stage 1 for the warp's NTW row tiles together: one Ub fragment load serves them all
      const float* xrow = xg + (size_t)q * (2 * E) + (size_t)(8 * wt + gq) * twoB;
      float dh[NTW][4], dl[NTW][4], dx[NTW][4];
      // An odd KS means a last k-step that holds the column b = B - 1 alone (a quarter of an MMA's K range): that
      // column is added with fp32 FMAs below instead, on the accumulator entries this lane owns.
      constexpr int KSM = (KS & 1) ? KS - 1 : KS;
#pragma unroll
      for (int ks = 0; ks < KSM; ++ks) {
        // Where a lane's float offset f lies past the row (the table holds zeros there) it reads the row's last
        // entry instead: finite data, no predicate.  KS odd means B = 4 (KS - 1) + 1: every step but the last is
        // whole, the last holds b = B - 1 alone.  KS == 8 means 16 <= B <= 32: the first four steps are whole.
        const int f = 32 * (ks >> 2) + 8 * t + 2 * (ks & 3);
        int fo;
        if ((KS & 1) && ks == KS - 1) fo = twoB - 2;
        else if ((KS & 1) || (KS == 8 && ks < 4)) fo = f;
        else fo = min(f, twoB - 2);
        const float4 uh = u1tab[ks * 32 + lane], ul = u1tab[(G.nbt + ks) * 32 + lane];
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          const float2 x = *reinterpret_cast<const float2*>(xrow + (size_t)(8 * nt * tw) * twoB + fo);
          float xh0, xl0, xh1, xl1;
          split_tf32_trunc(x.x, xh0, xl0); split_tf32_trunc(x.y, xh1, xl1);      // the streamed operand: cheapest split
          // A = (ur, -ui, ui, ur): rows (re, jb) and (im, jb) of W1
          if (ks == 0) {
            mma_tf32_z(dh[nt], uh.x, uh.y, uh.z, uh.w, xh0, xh1);
            mma_tf32_z(dl[nt], ul.x, ul.y, ul.z, ul.w, xh0, xh1);
            mma_tf32_z(dx[nt], uh.x, uh.y, uh.z, uh.w, xl0, xl1);
          } else {
            mma_tf32(dh[nt], uh.x, uh.y, uh.z, uh.w, xh0, xh1);
            mma_tf32(dl[nt], ul.x, ul.y, ul.z, ul.w, xh0, xh1);
            mma_tf32(dx[nt], uh.x, uh.y, uh.z, uh.w, xl0, xl1);
          }
        }
      }
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        // Y fragments: [0] Yre[a][jb], [1] Yre[a+1][jb], [2] Yim[a][jb], [3] Yim[a+1][jb], a = 8 tile + 2t, jb = gq
        float yh[4], yl[4];
        float ex[4] = {0.f, 0.f, 0.f, 0.f};
        if (KS & 1) {
          // Y[a][jb] += x[a][B-1] conj(Ub[B-1][jb]) for a = 8 tile + 2t, + 1 and jb = gq
          const float* xa = xg + (size_t)q * (2 * E) + (size_t)(8 * (wt + nt * tw) + 2 * t) * twoB + (twoB - 2);
          const float2 x0 = *reinterpret_cast<const float2*>(xa), x1 = *reinterpret_cast<const float2*>(xa + twoB);
          ex[0] = fmaf(x0.x, ulast.x, x0.y * ulast.y); ex[1] = fmaf(x1.x, ulast.x, x1.y * ulast.y);
          ex[2] = fmaf(x0.y, ulast.x, -x0.x * ulast.y); ex[3] = fmaf(x1.y, ulast.x, -x1.x * ulast.y);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) split_tf32((dh[nt][i] + ex[i]) + (dl[nt][i] + dx[nt][i]), yh[i], yl[i]);
#pragma unroll
        for (int mt = 0; mt < RAT; ++mt) {
          // (x, y, -y) of u0.hi, u1.hi, u0.lo, u1.lo with u0 = Ua[a][ja], u1 = Ua[a+1][ja]
          const float4 fh = ld_nc_f4_volatile(u2p[nt] + mt * 64), fl = ld_nc_f4_volatile(u2p[nt] + mt * 64 + 1);
          const float w[12] = {fh.x, fh.y, -fh.y, fh.z, fh.w, -fh.w, fl.x, fl.y, -fl.y, fl.z, fl.w, -fl.w};
          // step c = re: A = (u0.x, -u0.y, u1.x, -u1.y), B = (Yre[a], Yre[a+1]);  step c = im: A = (u0.y, u0.x, u1.y, u1.x)
          if (nt == 0) {
            mma_tf32_z(d2[mt][0], w[0], w[2], w[3], w[5], yh[0], yh[1]);
            mma_tf32_z(d2[mt][1], w[6], w[8], w[9], w[11], yh[0], yh[1]);
          } else {
            mma_tf32(d2[mt][0], w[0], w[2], w[3], w[5], yh[0], yh[1]);
            mma_tf32(d2[mt][1], w[6], w[8], w[9], w[11], yh[0], yh[1]);
          }
          mma_tf32(d2[mt][1], w[0], w[2], w[3], w[5], yl[0], yl[1]);
          mma_tf32(d2[mt][0], w[1], w[0], w[4], w[3], yh[2], yh[3]);
          mma_tf32(d2[mt][1], w[7], w[6], w[10], w[9], yh[2], yh[3]);
          mma_tf32(d2[mt][1], w[1], w[0], w[4], w[3], yl[2], yl[3]);
        }
      }
    } else {
#pragma unroll
      for (int mt = 0; mt < RAT; ++mt)
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 4; ++i) d2[mt][c][i] = 0.f;
    }
    // partial T of this warp's rows: row-major [8 RAT][8] complex, (d0, d2) = T[ja][2t], (d1, d3) = T[ja][2t+1]
    {
      float4* rw = reinterpret_cast<float4*>(red + ((size_t)(it & 1) * PJ_WARPS + warp) * REDW);
#pragma unroll
      for (int mt = 0; mt < RAT; ++mt)
        rw[4 * (8 * mt + gq) + t] = make_float4(d2[mt][0][0] + d2[mt][1][0], d2[mt][0][2] + d2[mt][1][2],
                                                d2[mt][0][1] + d2[mt][1][1], d2[mt][0][3] + d2[mt][1][3]);
    }
    // ---- off the critical path: the previous group's T, the next group's entries ----
    if (it > 0) reduce_out(u - gstride, it - 1);
    if (sparse) {
      // the zeroed entries were written through the generic proxy and a later bulk copy overwrites them: the
      // proxy fence of the writing threads can wait until here (the refill is issued after the next barrier)
      if (jcur < b1) fence_async_smem();
      b0 = c0; b1 = c1; pom = pomc;
      c0 = n0; c1 = n1;
      if (c0 + tid < c1) pomc = p.omega[c0 + tid];
    }
    pbuf = buf;
    if (++buf == nbuf) { buf = 0; phase ^= 1; }
  }
  if (it > 0) {
    __syncthreads();
    reduce_out(blockIdx.x + (it - 1) * gstride, it - 1);
  }
}

// ---------------------------------------------------------------------------------------------
// Reconstruction of the two trailing modes, fused with the weight update and the sparse add.
// Per slab W[A][B], with T'[ra][rb] the slab's tile of the partly reconstructed core; a warp
// owns 16 rows (am .. am+15) of one slab of the group:
//   stage 1  D1[a][(c,jb)] = sum_{(ja,c')} Ua[a][(ja,c')] Tt[(ja,c')][(c,jb)]    m16 = 16 rows a, n8 = 8 jb, one tile per c
//            step ks: k = t <-> (ja, re), k = t+4 <-> (ja, im), ja = 4 ks + t
//   stage 2  D [a][(b,c)]  = sum_{(jb,c')} Y'[a][(jb,c')] W3[(jb,c')][(b,c)]     m16 = 16 rows a, n8 = 4 complex b
//            step c': k = t <-> (jb, c'), k = t+4 <-> (jb+1, c'), jb = 2 t  (the accumulator layout of stage 1)
//            tile nb: n = g <-> (b, g & 1), b = 16 (nb>>2) + (nb&3) + 4 (g>>1), so lane (g, t) owns W[a][16 (nb>>2) + (nb&3) + 4 t]
// The sparse term is applied first (one entry per thread, scaled by 1/(1 - eta wd) so that the
// decayed dense update that follows leaves exactly eta*lambda*N_S), then each warp updates its
// rows in place and stores them with one bulk copy.
// ---------------------------------------------------------------------------------------------
// NBT > 0: the number of column tiles (tc_ksteps(B)) is built in and the loop over them unrolled; an odd NBT also
// fixes B = 4 (NBT - 1) + 1, so that every offset into a slab is an immediate.  NBT = 0: both at run time
template <int RAT, int NS, int NBT>
__global__ void __launch_bounds__(TC_THREADS, 2) back_tail_tc_kernel(void* __restrict__ w, TailTcParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  const TailParams& p = P.p;
  const TcGeom& G = P.g;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  const int B = (NBT & 1) ? 4 * (NBT - 1) + 1 : p.B, nbt = NBT ? NBT : G.nbt;
  const int ra = p.ra, rb = p.rb, twoB = 2 * B, nbuf = G.nbuf, spi = G.spi, tps = G.tps;
  const uint32_t E = p.E, nslab = p.nslab, ngroups = G.ngroups, gstride = gridDim.x;
  const int q = warp / tps, am = 16 * (warp - q * tps);
  const int r0 = am + gq, r1 = r0 + 8;
  constexpr int KS2 = 2 * RAT;
  float4* ubf = reinterpret_cast<float4*>(smem + G.off_aux);    // [nbt][2][32]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + G.off_bar);
  unsigned char* wb = static_cast<unsigned char*>(w);
  const int la = nbuf - 2;                                      // groups loaded ahead of the one being computed

  // Ua[r0][ja], Ua[r1][ja], ja = 4 ks + t: (u0.x, u1.x, u0.y, u1.y) hi, then lo
  float ua[KS2][8];
#pragma unroll
  for (int ks = 0; ks < KS2; ++ks) {
    const int ja = 4 * ks + t;
    cf v0 = (ja < ra) ? p.Ua[r0 * ra + ja] : make_float2(0.f, 0.f);
    cf v1 = (ja < ra) ? p.Ua[r1 * ra + ja] : make_float2(0.f, 0.f);
    cf h0, l0, h1, l1;
    split_tf32(v0.x, h0.x, l0.x); split_tf32(v0.y, h0.y, l0.y);
    split_tf32(v1.x, h1.x, l1.x); split_tf32(v1.y, h1.y, l1.y);
    ua[ks][0] = h0.x; ua[ks][1] = h1.x; ua[ks][2] = h0.y; ua[ks][3] = h1.y;
    ua[ks][4] = l0.x; ua[ks][5] = l1.x; ua[ks][6] = l0.y; ua[ks][7] = l1.y;
  }
  // Ub as stage-2 operand fragments, per column tile and lane:
  //   [nb][0][lane] = (b0re.hi, b1re.hi, b0re.lo, b1re.lo),  [nb][1][lane] = (b0im.hi, b1im.hi, b0im.lo, b1im.lo)
  //   step c' = re: W3[(jb,re)][(b,re)] = ur, [(b,im)] = ui;  step c' = im: [(b,re)] = -ui, [(b,im)] = ur
  for (int idx = tid; idx < nbt * 32; idx += TC_THREADS) {
    const int nb = idx >> 5, ln = idx & 31, g_ = ln >> 2, t_ = ln & 3;
    const int bq = 16 * (nb >> 2) + (nb & 3) + 4 * (g_ >> 1), jb = 2 * t_;
    const bool odd = g_ & 1;
    cf va = (bq < B && jb < rb) ? p.Ub[bq * rb + jb] : make_float2(0.f, 0.f);
    cf vb = (bq < B && jb + 1 < rb) ? p.Ub[bq * rb + jb + 1] : make_float2(0.f, 0.f);
    cf ah, al, bh, bl;
    split_tf32(va.x, ah.x, al.x); split_tf32(va.y, ah.y, al.y);
    split_tf32(vb.x, bh.x, bl.x); split_tf32(vb.y, bh.y, bl.y);
    ubf[(nb * 2 + 0) * 32 + ln] = odd ? make_float4(ah.y, bh.y, al.y, bl.y) : make_float4(ah.x, bh.x, al.x, bl.x);
    ubf[(nb * 2 + 1) * 32 + ln] = odd ? make_float4(ah.x, bh.x, al.x, bl.x) : make_float4(-ah.y, -bh.y, -al.y, -bl.y);
  }
  if (tid == 0) {
    for (int i = 0; i < nbuf; ++i) mbar_init(&bars[i], 1);
    fence_mbar_init();
  }
  __syncthreads();
  // Before the dependency wait: the operand tables above (Ua, Ub) and the first loads of W.  W was last written by
  // this kernel's launch of the previous step (or by the caller before this step), which completed before any
  // kernel of this step got past its own wait; nothing of this step writes it before this kernel does.
  if (tid == 0) {
    uint32_t u = blockIdx.x;
    for (int i = 0; i < la && u < ngroups; ++i, u += gstride) tc_issue_load(wb, smem, G, bars, u, i, nslab);
  }
  griddep_chain();
  const bool sparse = p.k > 0;
  int b0 = 0, b1 = 0, n0 = 0, n1 = 0;
  uint32_t pom = 0; cf pn = make_float2(0.f, 0.f);
  if (sparse) {
    uint32_t u = blockIdx.x;
    if (u < ngroups) {
      uint32_t e = (u + 1) * spi; if (e > nslab) e = nslab;
      b0 = (int)p.slab_ptr[u * spi]; b1 = (int)p.slab_ptr[e];
    }
    u += gstride;
    if (u < ngroups) {
      uint32_t e = (u + 1) * spi; if (e > nslab) e = nslab;
      n0 = (int)p.slab_ptr[u * spi]; n1 = (int)p.slab_ptr[e];
    }
    const int j = b0 + tid;
    if (j < b1) { pom = p.omega[j]; pn = p.n_s[j]; }
  }
  const bool decay = p.decay != 1.0f;
  const uint32_t row_bytes = 16u * (uint32_t)B * 8u;            // the 16 rows a warp owns
  uint32_t it = 0, phase = 0;
  int buf = 0, lbuf = la % nbuf;      // ring slot of this iteration and of the group loaded `la` ahead
  const int qstep = TC_WARPS / tps;      // this warp's NS slabs of a group are q, q + qstep, ...
  for (uint32_t u = blockIdx.x; u < ngroups; u += gstride, ++it) {
    if (lane == 0) bulk_wait_read<1>();     // this warp's stores of two iterations ago have read their rows
    // T' fragments for stage 1 (in flight while the slabs arrive): T'[ja = 4 ks + t][jb = gq]
    cf tv[NS][KS2];
#pragma unroll
    for (int i = 0; i < NS; ++i) {
      const uint32_t s = u * spi + q + i * qstep;
      const cf* tin = p.t + (size_t)s * ra * rb;
#pragma unroll
      for (int ks = 0; ks < KS2; ++ks) {
        const int ja = 4 * ks + t;
        tv[i][ks] = (s < nslab && ja < ra && gq < rb) ? __ldg(tin + (size_t)ja * rb + gq) : make_float2(0.f, 0.f);
      }
    }
    const bool ok = mbar_wait_bounded(&bars[buf], phase);
    float* wg = reinterpret_cast<float*>(smem + (size_t)buf * G.grp_stride);
    // ---- scaled sparse add at Omega, one entry of the group per thread ----
    if (sparse && ok) {
      const uint32_t base = u * (uint32_t)spi * E;
      int j = b0 + tid;
      if (j < b1) {
        cf* wp = reinterpret_cast<cf*>(wg) + (pom - base);
        cf wv = *wp;
        wv.x = fmaf(-P.s_sparse_pre, pn.x, wv.x); wv.y = fmaf(-P.s_sparse_pre, pn.y, wv.y);
        *wp = wv;
      }
      for (j += TC_THREADS; j < b1; j += TC_THREADS) {
        cf* wp = reinterpret_cast<cf*>(wg) + (p.omega[j] - base);
        cf n = p.n_s[j];
        cf wv = *wp;
        wv.x = fmaf(-P.s_sparse_pre, n.x, wv.x); wv.y = fmaf(-P.s_sparse_pre, n.y, wv.y);
        *wp = wv;
      }
      b0 = n0; b1 = n1;
      j = b0 + tid;
      if (j < b1) { pom = p.omega[j]; pn = p.n_s[j]; }
      const uint32_t u3 = u + 2 * gstride;
      n0 = n1 = 0;
      if (u3 < ngroups) {
        uint32_t e = (u3 + 1) * spi; if (e > nslab) e = nslab;
        n0 = (int)p.slab_ptr[u3 * spi]; n1 = (int)p.slab_ptr[e];
      }
    }
    if (__syncthreads_or(!ok)) {
      if (tid == 0) {
        atomicOr(P.flags, 4);
        uint32_t ux = u + gstride, ph = phase;
        int bx = buf;
        for (int i = 1; i < la && ux < ngroups; ++i, ux += gstride) {
          if (++bx == nbuf) { bx = 0; ph ^= 1; }
          mbar_wait_bounded(&bars[bx], ph, 1u << 16);
        }
      }
      if (lane == 0) bulk_wait_all<0>();
      return;
    }
    // every warp's store of iteration it-2 has been read (checked before the barrier): its buffer takes group it+la
    if (tid == 0) {
      const uint32_t un = u + (uint32_t)la * gstride;
      if (un < ngroups) tc_issue_load(wb, smem, G, bars, un, lbuf, nslab);
    }
#pragma unroll
    for (int i = 0; i < NS; ++i) {
    const int qi = q + i * qstep;
    const uint32_t s = u * spi + qi;
    const bool active = s < nslab;
    if (active) {
      float* ws = wg + (size_t)qi * (2 * E);
      // ---- stage 1: Y'[a][(c, jb)] for rows r0 and r1; hi*hi, lo*hi and hi*lo accumulate separately ----
      float d1[2][3][4];
#pragma unroll
      for (int ks = 0; ks < KS2; ++ks) {
        float trh, trl, tih, til;
        split_tf32(tv[i][ks].x, trh, trl); split_tf32(tv[i][ks].y, tih, til);
        const float* a = ua[ks];
        // A = (Ua[r0].re, Ua[r1].re, Ua[r0].im, Ua[r1].im);  re tile: B = (Tr, -Ti);  im tile: B = (Ti, Tr)
        if (ks == 0) {
          mma_tf32_z(d1[0][0], a[0], a[1], a[2], a[3], trh, -tih);
          mma_tf32_z(d1[0][1], a[4], a[5], a[6], a[7], trh, -tih);
          mma_tf32_z(d1[0][2], a[0], a[1], a[2], a[3], trl, -til);
          mma_tf32_z(d1[1][0], a[0], a[1], a[2], a[3], tih, trh);
          mma_tf32_z(d1[1][1], a[4], a[5], a[6], a[7], tih, trh);
          mma_tf32_z(d1[1][2], a[0], a[1], a[2], a[3], til, trl);
        } else {
          mma_tf32(d1[0][0], a[0], a[1], a[2], a[3], trh, -tih);
          mma_tf32(d1[0][1], a[4], a[5], a[6], a[7], trh, -tih);
          mma_tf32(d1[0][2], a[0], a[1], a[2], a[3], trl, -til);
          mma_tf32(d1[1][0], a[0], a[1], a[2], a[3], tih, trh);
          mma_tf32(d1[1][1], a[4], a[5], a[6], a[7], tih, trh);
          mma_tf32(d1[1][2], a[0], a[1], a[2], a[3], til, trl);
        }
      }
      // Y' as stage-2 A fragments: a0 = d[0] (row g, jb), a1 = d[2] (row g+8, jb), a2 = d[1] (row g, jb+1), a3 = d[3]
      float yh[2][4], yl[2][4];
#pragma unroll
      for (int c = 0; c < 2; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i) split_tf32(d1[c][0][i] + (d1[c][1][i] + d1[c][2][i]), yh[c][i], yl[c][i]);
      // ---- stage 2, one column tile at a time, applied to the slab right away ----
      float* w0row = ws + (size_t)r0 * twoB;
      float* w1row = ws + (size_t)r1 * twoB;
      constexpr int NB_UNROLL = NBT ? NBT : 3;
#pragma unroll NB_UNROLL
      for (int nb = 0; nb < nbt; ++nb) {
        const float4 fr = ubf[(nb * 2 + 0) * 32 + lane], fi = ubf[(nb * 2 + 1) * 32 + lane];
        float dh[4], dl[4], dx[4];
        mma_tf32_z(dh, yh[0][0], yh[0][2], yh[0][1], yh[0][3], fr.x, fr.y);
        mma_tf32_z(dl, yl[0][0], yl[0][2], yl[0][1], yl[0][3], fr.x, fr.y);
        mma_tf32_z(dx, yh[0][0], yh[0][2], yh[0][1], yh[0][3], fr.z, fr.w);
        mma_tf32(dh, yh[1][0], yh[1][2], yh[1][1], yh[1][3], fi.x, fi.y);
        mma_tf32(dl, yl[1][0], yl[1][2], yl[1][1], yl[1][3], fi.x, fi.y);
        mma_tf32(dx, yh[1][0], yh[1][2], yh[1][1], yh[1][3], fi.z, fi.w);
        // d0 + i d1 = D[r0][b], d2 + i d3 = D[r1][b] with b = 16 (nb>>2) + (nb&3) + 4 t
        const int bo = 16 * (nb >> 2) + (nb & 3) + 4 * t;
        if (bo < B) {
          float2* p0 = reinterpret_cast<float2*>(w0row) + bo;
          float2* p1 = reinterpret_cast<float2*>(w1row) + bo;
          float2 v0 = *p0, v1 = *p1;
          if (decay) { v0.x *= p.decay; v0.y *= p.decay; v1.x *= p.decay; v1.y *= p.decay; }
          v0.x = fmaf(-p.s_low, dh[0] + (dl[0] + dx[0]), v0.x); v0.y = fmaf(-p.s_low, dh[1] + (dl[1] + dx[1]), v0.y);
          v1.x = fmaf(-p.s_low, dh[2] + (dl[2] + dx[2]), v1.x); v1.y = fmaf(-p.s_low, dh[3] + (dl[3] + dx[3]), v1.y);
          *p0 = v0; *p1 = v1;
        }
      }
    }
    fence_async_smem();     // order this lane's shared-memory writes before the bulk store reads them
    __syncwarp();
    if (lane == 0 && active)
      bulk_s2g(wb + ((size_t)s * E + (size_t)am * B) * 8, smem + (size_t)buf * G.grp_stride + (size_t)qi * G.slab_bytes +
                                                              (size_t)am * B * 8, row_bytes);
    }
    if (lane == 0) bulk_commit();      // one group per iteration, whatever it holds
    if (++buf == nbuf) { buf = 0; phase ^= 1; }
    if (++lbuf == nbuf) lbuf = 0;
  }
  if (lane == 0) bulk_wait_all<0>();   // stores complete before the block's shared memory goes away
}

}  // namespace tg
