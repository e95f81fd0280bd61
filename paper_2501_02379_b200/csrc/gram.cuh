// Mode-n Gram matrices of the residual, A_n = R_(n) R_(n)^H (I_n x I_n,
// Hermitian PSD), from which the factor matrices are refreshed
// (TuckerFactors of Algorithm 1: leading left singular vectors of the mode-n
// unfolding = leading eigenvectors of A_n).  The Gram matrix does not depend on
// the column order of the unfolding, so the tensor is read in place as
// [O][I_n][C] with C contiguous.
//
// Only tile pairs on or above the diagonal are computed; split-K partial sums
// go to scratch and are reduced in a fixed order (deterministic result).
#pragma once
#include "common.cuh"

namespace tg {

constexpr int GR_T = 64;     // output tile (rows a x cols b)
constexpr int GR_KT = 16;    // K chunk
constexpr int GR_LD = 66;    // padded tile row length in shared memory (keeps 16-byte alignment)

template <class S>
__global__ void __launch_bounds__(256) gram_partial_kernel(const void* __restrict__ g, int In, uint32_t O, uint32_t C,
                                                           uint32_t chunks_total, uint32_t chunks_per_split,
                                                           cf* __restrict__ partial) {
  const int T = (In + GR_T - 1) / GR_T;
  const int ta = blockIdx.x / T, tb = blockIdx.x % T;
  if (ta > tb) return;
  __shared__ __align__(16) cf Xa[GR_KT][GR_LD];
  __shared__ __align__(16) cf Xb[GR_KT][GR_LD];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int a0 = ta * GR_T, b0 = tb * GR_T;
  const uint32_t cpo = (C + GR_KT - 1) / GR_KT;   // chunks per o when C > 1
  uint32_t ch0 = blockIdx.y * chunks_per_split;
  uint32_t ch1 = ch0 + chunks_per_split; if (ch1 > chunks_total) ch1 = chunks_total;
  cf acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = make_float2(0.f, 0.f);

  for (uint32_t ch = ch0; ch < ch1; ++ch) {
    if (C == 1) {
      // last mode: K index is o itself, rows of the tile are contiguous in memory
      const uint32_t o0 = ch * GR_KT;
      for (int i = tid; i < GR_KT * GR_T; i += 256) {
        int aa = i % GR_T, kk = i / GR_T;
        uint32_t o = o0 + kk;
        cf va = make_float2(0.f, 0.f), vb = va;
        if (o < O) {
          if (a0 + aa < In) va = S::load(g, (size_t)o * In + a0 + aa);
          if (b0 + aa < In) vb = S::load(g, (size_t)o * In + b0 + aa);
        }
        Xa[kk][aa] = va; Xb[kk][aa] = vb;
      }
    } else {
      const uint32_t o = ch / cpo, c0 = (ch - o * cpo) * GR_KT;
      for (int i = tid; i < GR_KT * GR_T; i += 256) {
        int kk = i % GR_KT, aa = i / GR_KT;
        uint32_t c = c0 + kk;
        cf va = make_float2(0.f, 0.f), vb = va;
        if (c < C) {
          if (a0 + aa < In) va = S::load(g, ((size_t)o * In + a0 + aa) * C + c);
          if (b0 + aa < In) vb = S::load(g, ((size_t)o * In + b0 + aa) * C + c);
        }
        Xa[kk][aa] = va; Xb[kk][aa] = vb;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < GR_KT; ++kk) {
      float4 p0 = *reinterpret_cast<const float4*>(&Xa[kk][ty * 4]);
      float4 p1 = *reinterpret_cast<const float4*>(&Xa[kk][ty * 4 + 2]);
      float4 q0 = *reinterpret_cast<const float4*>(&Xb[kk][tx * 4]);
      float4 q1 = *reinterpret_cast<const float4*>(&Xb[kk][tx * 4 + 2]);
      cf a[4] = {make_float2(p0.x, p0.y), make_float2(p0.z, p0.w), make_float2(p1.x, p1.y), make_float2(p1.z, p1.w)};
      cf b[4] = {make_float2(q0.x, q0.y), make_float2(q0.z, q0.w), make_float2(q1.x, q1.y), make_float2(q1.z, q1.w)};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) cfma_conj(acc[i][j], a[i], b[j]);
    }
    __syncthreads();
  }
  cf* out = partial + (size_t)blockIdx.y * In * In;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int a = a0 + ty * 4 + i;
    if (a >= In) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int b = b0 + tx * 4 + j;
      if (b < In) out[(size_t)a * In + b] = acc[i][j];
    }
  }
}

// Sum the split-K partials in split order; mirror the upper triangle.
__global__ void gram_reduce_kernel(const cf* __restrict__ partial, int splits, int In, cf* __restrict__ A) {
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= In * In) return;
  int a = idx / In, b = idx % In;
  if (a > b) return;
  float sx = 0.f, sy = 0.f;
  for (int s = 0; s < splits; ++s) {
    cf v = partial[(size_t)s * In * In + idx];
    sx += v.x; sy += v.y;
  }
  if (a == b) { A[idx] = make_float2(sx, 0.f); return; }
  A[idx] = make_float2(sx, sy);
  A[(size_t)b * In + a] = make_float2(sx, -sy);
}

}  // namespace tg
