// Mode-n Gram matrices of the residual, A_n = R_(n) R_(n)^H (I_n x I_n,
// Hermitian PSD), from which the factor matrices are refreshed
// (TuckerFactors of Algorithm 1: leading left singular vectors of the mode-n
// unfolding = leading eigenvectors of A_n).  The Gram matrix does not depend on
// the column order of the unfolding, so the tensor is read in place as
// [O][I_n][C] with C contiguous and the contraction index k = (o, c) flattened.
//
// Tensor cores, TF32 inputs, fp32 accumulation.  With rows as interleaved real
// vectors X'[a] = (re, im, re, im, ...):
//   Re A[a][b] = X'[a] . X'[b],   Im A[a][b] = X'[a] . Y'[b],  Y'[b] = (-im, re, -im, re, ...)
// so one loaded fragment of row b serves both products.  A block owns a 64 x 64
// tile of A (only tiles on or above the diagonal are computed), a warp 32 x 32
// of it; K is split over blockIdx.y, partial sums go to scratch and are reduced
// in a fixed order (deterministic result).
// SPLIT = false: inputs rounded to TF32 once (relative error of an entry of A about
// 2^-11.5 / sqrt(K) of the diagonal scale: used when K is large).  SPLIT = true:
// x = hi + lo and the three products hi*hi, hi*lo, lo*hi (fp32-grade, for short K).
#pragma once
#include "common.cuh"
#include "ptx.cuh"

namespace tg {

constexpr int GR_T = 64;      // output tile (rows a x cols b)
constexpr int GR_KT = 32;     // complex k per shared-memory chunk
constexpr int GR_LD = 36;     // padded chunk row length: fragment loads (8 rows x 4 k) hit distinct banks
constexpr int GR_THREADS = 128;

__device__ __forceinline__ float gr_tf32(float x) { return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u); }

constexpr size_t GR_SMEM = 2 * 2 * GR_T * GR_LD * sizeof(cf);      // two stages of (Xa, Xb)

// FULL: I_n is a multiple of the tile, so no sub-tile of a warp is empty and the MMA loop has no branches
template <class S, bool SPLIT, bool FULL>
__global__ void __launch_bounds__(GR_THREADS, 3) gram_partial_kernel(const void* __restrict__ g, int In, uint32_t O, uint32_t C,
                                                                  uint32_t chunks_total, uint32_t chunks_per_split,
                                                                  cf* __restrict__ partial) {
  const int T = (In + GR_T - 1) / GR_T;
  const int ta = blockIdx.x / T, tb = blockIdx.x % T;
  if (ta > tb) return;
  extern __shared__ __align__(16) unsigned char gsm[];
  // tiles hold the entries as they are stored (fp32 pairs, or fp16 / bfloat16 pairs in one word): 16-bit values are
  // exact TF32 operands, so 16-bit storage needs neither rounding nor the split products
  typedef typename S::elem Elem;
  typedef Elem Tile[GR_T][GR_LD];
  Tile* XA = reinterpret_cast<Tile*>(gsm);            // [2]
  Tile* XBs = XA + 2;                                 // [2]
  constexpr bool HALF = S::kBytes == 4;
  constexpr bool DOSPLIT = SPLIT && !HALF;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, t = lane & 3;
  // 2 x 2 warps of 32 x 32.  A matrix of at most 32 rows lies in the first warp's quarter alone: the four warps then
  // all take that quarter and share the contraction range instead (k-step ks goes to warp ks mod 4), and their sums are
  // added at the end.
  const bool ksplit = In <= 32;
  const int wm = ksplit ? 0 : warp >> 1, wn = ksplit ? 0 : warp & 1;
  const int a0 = ta * GR_T, b0 = tb * GR_T;
  const bool diag = ta == tb;
  const uint32_t K32 = O * C;                        // the tensor has fewer than 2^32 entries
  uint32_t ch0 = blockIdx.y * chunks_per_split;
  uint32_t ch1 = ch0 + chunks_per_split; if (ch1 > chunks_total) ch1 = chunks_total;
  // which 16-row / 8-column sub-tiles of this warp hold any row of A
  bool mok[2], nok[4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) mok[mt] = FULL || a0 + wm * 32 + mt * 16 < In;
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) nok[nt] = FULL || b0 + wn * 32 + nt * 8 < In;
  float are[2][4][4], aim[2][4][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) { are[mt][nt][i] = 0.f; aim[mt][nt][i] = 0.f; }
  // The tensor core adds into its fp32 accumulator with truncation, which biases a long chain of
  // accumulations; so the MMA accumulators are emptied every other chunk (16 MMAs deep) into
  // running sums kept with ordinary round-to-nearest adds.
  float tre[2][4][4], tim[2][4][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) { tre[mt][nt][i] = 0.f; tim[mt][nt][i] = 0.f; }
  // Loader.  Rows of a tile beyond the matrix are never loaded: the tiles are zeroed once, and only the rows that
  // exist are copied (the copies of a chunk's entries beyond the contraction range write zeros).  Rows are runs of
  // k (C > 1): a thread keeps one k of the chunk and walks the existing rows, four apart.  C == 1 (the rows of one k
  // are contiguous): the threads are spread over (existing rows) x (as many k as that leaves room for).
  const bool along_k = C > 1;
  const int nra = min(GR_T, In - a0), nrb = min(GR_T, In - b0);            // rows of the two tiles that exist
  const int ld_kc = tid % GR_KT, ld_row = tid / GR_KT;                     // C > 1
  const int ka = GR_THREADS / nra, kb = GR_THREADS / nrb;                  // C == 1: k per pass (at least 2)
  const int ra1 = tid % nra, ka0 = tid / nra, rb1 = tid % nrb, kb0 = tid / nrb;
  const unsigned char* gb = static_cast<const unsigned char*>(g);
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(gsm);
    for (int idx = tid; idx < (int)(GR_SMEM / 4); idx += GR_THREADS) z[idx] = 0u;
    __syncthreads();
  }
  auto copy1 = [&](Elem* dst, size_t entry, bool ok) {
    if (!HALF) cp_async8(dst, ok ? gb + entry * 8 : gb, ok ? 8u : 0u);
    else cp_async4(dst, ok ? gb + entry * 4 : gb, ok ? 4u : 0u);
  };

  // chunk ch -> stage st: asynchronous 8-byte (fp32 storage) or 4-byte (16-bit storage) copies
  auto load_chunk = [&](uint32_t ch, int st) {
    const uint32_t kk0 = ch * GR_KT;
    Elem (*xa)[GR_LD] = XA[st];
    Elem (*xb)[GR_LD] = XBs[st];
    if (along_k) {
      const uint32_t kk = kk0 + ld_kc;
      const bool kok = kk < K32;
      const uint32_t o = kok ? kk / C : 0, c = kok ? kk - o * C : 0;
      const size_t base = (size_t)o * In * C + c;
      for (int row = ld_row; row < nra; row += GR_THREADS / GR_KT) copy1(&xa[row][ld_kc], base + (size_t)(a0 + row) * C, kok);
      if (!diag)
        for (int row = ld_row; row < nrb; row += GR_THREADS / GR_KT) copy1(&xb[row][ld_kc], base + (size_t)(b0 + row) * C, kok);
    } else {
      if (ka0 < ka)
        for (int kc = ka0; kc < GR_KT; kc += ka) copy1(&xa[ra1][kc], (size_t)(kk0 + kc) * In + a0 + ra1, kk0 + kc < K32);
      if (!diag && kb0 < kb)
        for (int kc = kb0; kc < GR_KT; kc += kb) copy1(&xb[rb1][kc], (size_t)(kk0 + kc) * In + b0 + rb1, kk0 + kc < K32);
    }
    cp_async_commit();
  };

  if (ch0 < ch1) load_chunk(ch0, 0);
  int st = 0;
  for (uint32_t ch = ch0; ch < ch1; ++ch, st ^= 1) {
    cp_async_wait<0>();
    __syncthreads();                                   // chunk ch has landed; everyone is done with stage st^1
    if (ch + 1 < ch1) load_chunk(ch + 1, st ^ 1);
    const Elem (*Xa)[GR_LD] = XA[st];
    const Elem (*XB)[GR_LD] = diag ? XA[st] : XBs[st];
    auto widen = [](const Elem& e) -> cf {
      return S::widen(e);
    };
    if (HALF) {
      // 16-bit storage: a stored (re, im) pair is one packed operand register of the m16n8k16 shape (k = 2c, 2c + 1),
      // so the tiles are contracted as stored, exactly, eight entries per instruction; y = (-im, re) is a swap of
      // the halves and a sign flip
      const uint32_t (*Ua)[GR_LD] = reinterpret_cast<const uint32_t (*)[GR_LD]>(Xa);
      const uint32_t (*Ub)[GR_LD] = reinterpret_cast<const uint32_t (*)[GR_LD]>(XB);
#pragma unroll
      for (int ks = 0; ks < GR_KT / 8; ++ks) {
        if (ksplit && (ks & 3) != warp) continue;
        const int kc = ks * 8 + t;
        uint32_t a[2][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          const int r = wm * 32 + mt * 16 + gq;
          a[mt][0] = Ua[r][kc]; a[mt][1] = Ua[r + 8][kc]; a[mt][2] = Ua[r][kc + 4]; a[mt][3] = Ua[r + 8][kc + 4];
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          if (!FULL && !nok[nt]) continue;
          const int r = wn * 32 + nt * 8 + gq;
          const uint32_t b0 = Ub[r][kc], b1 = Ub[r][kc + 4];
          const uint32_t y0 = ((b0 >> 16) ^ 0x8000u) | (b0 << 16), y1 = ((b1 >> 16) ^ 0x8000u) | (b1 << 16);
#pragma unroll
          for (int mt = 0; mt < 2; ++mt) {
            if (!FULL && !mok[mt]) continue;
            if (S::kBf16) {
              mma_bf16(are[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b0, b1);
              mma_bf16(aim[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], y0, y1);
            } else {
              mma_f16(are[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], b0, b1);
              mma_f16(aim[mt][nt], a[mt][0], a[mt][1], a[mt][2], a[mt][3], y0, y1);
            }
          }
        }
      }
    } else
#pragma unroll
    for (int ks = 0; ks < GR_KT / 4; ++ks) {
      if (ksplit && (ks & 3) != warp) continue;
      const int kc = ks * 4 + t;
      // A fragments: (row g, re), (row g+8, re), (row g, im), (row g+8, im)
      float ah[2][4], al[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        const cf x0 = widen(Xa[wm * 32 + mt * 16 + gq][kc]), x1 = widen(Xa[wm * 32 + mt * 16 + gq + 8][kc]);
        if (HALF) { ah[mt][0] = x0.x; ah[mt][1] = x1.x; ah[mt][2] = x0.y; ah[mt][3] = x1.y; }
        else { ah[mt][0] = gr_tf32(x0.x); ah[mt][1] = gr_tf32(x1.x); ah[mt][2] = gr_tf32(x0.y); ah[mt][3] = gr_tf32(x1.y); }
        if (DOSPLIT) { al[mt][0] = x0.x - ah[mt][0]; al[mt][1] = x1.x - ah[mt][1]; al[mt][2] = x0.y - ah[mt][2]; al[mt][3] = x1.y - ah[mt][3]; }
      }
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        if (!FULL && !nok[nt]) continue;
        const cf y = widen(XB[wn * 32 + nt * 8 + gq][kc]);
        const float yh0 = HALF ? y.x : gr_tf32(y.x), yh1 = HALF ? y.y : gr_tf32(y.y);
        const float yl0 = y.x - yh0, yl1 = y.y - yh1;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
          if (!FULL && !mok[mt]) continue;
          mma_tf32(are[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], yh0, yh1);
          mma_tf32(aim[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], -yh1, yh0);
          if (DOSPLIT) {
            mma_tf32(are[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], yl0, yl1);
            mma_tf32(aim[mt][nt], ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3], -yl1, yl0);
            mma_tf32(are[mt][nt], al[mt][0], al[mt][1], al[mt][2], al[mt][3], yh0, yh1);
            mma_tf32(aim[mt][nt], al[mt][0], al[mt][1], al[mt][2], al[mt][3], -yh1, yh0);
          }
        }
      }
    }
    if (((ch - ch0) & 1) || ch + 1 == ch1) {
#pragma unroll
      for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            tre[mt][nt][i] += are[mt][nt][i]; are[mt][nt][i] = 0.f;
            tim[mt][nt][i] += aim[mt][nt][i]; aim[mt][nt][i] = 0.f;
          }
    }
  }
  if (ksplit) {
    // the four warps' sums of the same quarter, added in a fixed order by the first warp (through the tile memory)
    __syncthreads();
    float* red = reinterpret_cast<float*>(gsm);          // [warp][re|im][mt][nt][i][lane]: 32 KB
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          red[((((warp * 2 + 0) * 2 + mt) * 4 + nt) * 4 + i) * 32 + lane] = tre[mt][nt][i];
          red[((((warp * 2 + 1) * 2 + mt) * 4 + nt) * 4 + i) * 32 + lane] = tim[mt][nt][i];
        }
    __syncthreads();
    if (warp != 0) return;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float sr = 0.f, si = 0.f;
          for (int w = 0; w < 4; ++w) {
            sr += red[((((w * 2 + 0) * 2 + mt) * 4 + nt) * 4 + i) * 32 + lane];
            si += red[((((w * 2 + 1) * 2 + mt) * 4 + nt) * 4 + i) * 32 + lane];
          }
          tre[mt][nt][i] = sr; tim[mt][nt][i] = si;
        }
  }
  // accumulator (row g | g+8, col 2t | 2t+1) -> partial[split][a][b]
  cf* out = partial + (size_t)blockIdx.y * In * In;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int a = a0 + wm * 32 + mt * 16 + gq + (i >> 1) * 8, b = b0 + wn * 32 + nt * 8 + 2 * t + (i & 1);
        if (a < In && b < In) out[(size_t)a * In + b] = make_float2(tre[mt][nt][i], tim[mt][nt][i]);
      }
}

// Sum the split-K partials, always in the same order (sixteen interleaved running sums per entry, then
// those in order): deterministic.  Mirrors the upper triangle.
constexpr int GRR_E = 64, GRR_G = 16;    // entries per block, split groups
__global__ void __launch_bounds__(GRR_E * GRR_G) gram_reduce_kernel(const cf* __restrict__ partial, int splits, int In,
                                                                   cf* __restrict__ A) {
  __shared__ cf part[GRR_G][GRR_E];
  const int e = threadIdx.x % GRR_E, sg = threadIdx.x / GRR_E;
  const int idx = blockIdx.x * GRR_E + e;
  const int n2 = In * In;
  const int a = idx < n2 ? idx / In : 0, b = idx < n2 ? idx - a * In : 0;
  const bool live = idx < n2 && a <= b;
  float sx = 0.f, sy = 0.f;
  if (live) {
    const cf* p = partial + idx;
#pragma unroll 4
    for (int s = sg; s < splits; s += GRR_G) {
      cf v = p[(size_t)s * n2];
      sx += v.x; sy += v.y;
    }
  }
  part[sg][e] = make_float2(sx, sy);
  __syncthreads();
  if (sg == 0 && live) {
    for (int q = 1; q < GRR_G; ++q) { sx += part[q][e].x; sy += part[q][e].y; }
    if (a == b) { A[idx] = make_float2(sx, 0.f); return; }
    A[idx] = make_float2(sx, sy);
    A[(size_t)b * In + a] = make_float2(sx, -sy);
  }
}

}  // namespace tg
