// Magnitude top-k selection of the sparse index set Omega
// (SparseIndices with the top-k strategy, Section 2.2 "Unstructured sparse
// gradient tensor"): radix select on the fp32 bit pattern of |g|^2 (first digit on the tensor, the other two on a
// copy of the threshold bucket's keys), then an ordered compaction that writes Omega ascending.  Ties at the threshold key
// go to the lower flat index.  Everything is integer work after the key, and
// no result depends on the order in which atomics land.
#pragma once
#include "common.cuh"

namespace tg {

struct SelState {
  uint32_t prefix;   // key bits fixed so far (high bits)
  uint32_t krem;     // rank still to resolve inside the current prefix bucket
  uint32_t thr;      // final threshold key (valid after the last pass)
  uint32_t take_eq;  // how many entries with key == thr belong to Omega
  // After the first pass only the keys of the threshold bucket matter.  When they fit the candidate buffer they are
  // copied there (one more pass over the tensor, which also counts, per block of kChunk entries, the keys above the
  // bucket), the second and third digit are found on the copy, and the per-block counts are completed from it: three
  // passes over the tensor (histogram, copy, compaction) instead of five.
  uint32_t cand_cap;    // capacity of the candidate buffer in keys (0: never used)
  uint32_t use_cand;    // decided by the first pick
  uint32_t cand_total;  // keys in the buffer
  uint32_t pad;
};

// What the entries are ranked by (SparseIndices of Algorithm 1 with one of the sparsification strategies of
// Section 2.2): 0 top-k magnitude, 1 uniform random selection, 2 probabilistic sampling proportional to |g|.
struct SelKey {
  uint32_t seed_lo, seed_hi;   // key of the counter-based generator
  uint32_t epoch;              // number of the refresh (the sets are redrawn at every refresh)
  int strategy;
};

// First output word of Philox-4x32 with 10 rounds (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3") for
// the counter (i, epoch, 0, 0).
__device__ __forceinline__ uint32_t sel_word(uint32_t i, const SelKey& kp) {
  uint32_t c0 = i, c1 = kp.epoch, c2 = 0u, c3 = 0u, k0 = kp.seed_lo, k1 = kp.seed_hi;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), l0 = 0xD2511F53u * c0;
    const uint32_t h1 = __umulhi(0xCD9E8D57u, c2), l1 = 0xCD9E8D57u * c2;
    c0 = h1 ^ c1 ^ k0; c1 = l1; c2 = h0 ^ c3 ^ k1; c3 = l0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

// E = -ln(u), u = ((word >> 9) + 1/2) 2^-23: a unit-rate exponential variate.  A fixed sequence of IEEE fp32
// operations without fused multiply-adds, so that any implementation of the same recipe gets the same bits:
// u = m 2^e with m in (sqrt(1/2), sqrt(2)], f = m - 1, s = f / (f + 2), z = s s,
// ln m = 2 (s + s z (1/3 + z (1/5 + z (1/7 + z / 9)))), ln u = e ln 2 + ln m.
__device__ __forceinline__ float sel_neg_log(uint32_t word) {
  const float u = __fmul_rn(__fadd_rn((float)(word >> 9), 0.5f), 1.1920928955078125e-07f);   // 2^-23
  const uint32_t bits = __float_as_uint(u);
  int e = (int)(bits >> 23) - 127;
  float m = __uint_as_float((bits & 0x7FFFFFu) | 0x3F800000u);
  if (m > 1.41421354f) { m = __fmul_rn(m, 0.5f); e += 1; }
  const float f = __fadd_rn(m, -1.0f);
  const float sq = __fdiv_rn(f, __fadd_rn(f, 2.0f));
  const float z = __fmul_rn(sq, sq);
  float pl = __fmul_rn(0.111111112f, z);
  pl = __fadd_rn(pl, 0.142857149f);
  pl = __fmul_rn(pl, z);
  pl = __fadd_rn(pl, 0.2f);
  pl = __fmul_rn(pl, z);
  pl = __fadd_rn(pl, 0.333333343f);
  float r = __fmul_rn(sq, z);
  r = __fmul_rn(r, pl);
  r = __fadd_rn(r, sq);
  r = __fmul_rn(r, 2.0f);
  float ln_u = __fmul_rn((float)e, 0.693147182f);
  ln_u = __fadd_rn(ln_u, r);
  return -ln_u;
}

// The key of entry i with value v: its k largest (ties to the lower index) are selected.  Keys are non-negative
// floats or plain integers, so their bit patterns order like their values.
__device__ __forceinline__ uint32_t sel_key(cf v, uint32_t i, const SelKey& kp) {
  if (kp.strategy == 0) return mag_key(v);
  const uint32_t w = sel_word(i, kp);
  if (kp.strategy == 1) return w;
  const float mag = __fsqrt_rn(__uint_as_float(mag_key(v)));
  return __float_as_uint(__fdiv_rn(mag, sel_neg_log(w)));
}

// three passes over the 32 key bits: 11 + 11 + 10
__host__ __device__ inline int sel_bits(int pass) { return pass == 2 ? 10 : 11; }
__host__ __device__ inline int sel_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
constexpr int kSelMaxBins = 2048;
constexpr int kChunk = 2048;        // elements per compaction block
constexpr int kChunkThreads = 256;  // 8 consecutive elements per thread

__global__ void sel_init_kernel(SelState* st, uint32_t k, uint32_t cand_cap) {
  st->prefix = 0u; st->krem = k; st->thr = 0u; st->take_eq = 0u;
  st->cand_cap = cand_cap; st->use_cand = 0u; st->cand_total = 0u; st->pad = 0u;
}

// Histogram of the current digit over all entries whose higher bits equal the
// prefix chosen so far.
// TOPK: the key is the magnitude (the strategy of Algorithm 1 and of the five benchmark configurations): built in, so
// that this path carries nothing of the random strategies.
template <class S, bool TOPK>
__global__ void __launch_bounds__(512) sel_hist_kernel(const void* __restrict__ g, uint32_t n, int pass,
                                                      const SelState* __restrict__ st, uint32_t* __restrict__ hist,
                                                      int* __restrict__ flags, SelKey kp) {
  __shared__ uint32_t sh[kSelMaxBins];
  if (pass > 0 && st->use_cand) return;        // the later digits come from the candidate buffer
  const int bits = sel_bits(pass), shift = sel_shift(pass);
  const uint32_t nb = 1u << bits;
  for (uint32_t i = threadIdx.x; i < nb; i += blockDim.x) sh[i] = 0u;
  __syncthreads();
  const uint32_t prefix = st->prefix;
  const uint32_t hi_mask = (pass == 0) ? 0u : (0xffffffffu << (shift + bits));
  bool bad = false;
  constexpr int UN = 4;                       // entries per thread and iteration: their loads are issued together
  const uint64_t stride = (uint64_t)gridDim.x * blockDim.x * UN;
  for (uint64_t b0 = (uint64_t)blockIdx.x * blockDim.x * UN; b0 < n; b0 += stride) {
    uint32_t keys[UN];
    bool valid[UN];
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const uint64_t i = b0 + (uint64_t)j * blockDim.x + threadIdx.x;
      valid[j] = i < n;
      cf v = make_float2(0.f, 0.f);
      if (valid[j]) v = S::load(g, i);
      keys[j] = valid[j] ? (TOPK ? mag_key(v) : sel_key(v, (uint32_t)i, kp)) : 0u;
      // a NaN or an infinity among the magnitudes (the random strategy does not look at them)
      if (pass == 0 && (TOPK || kp.strategy != 1) && (mag_key(v) & 0x7f800000u) == 0x7f800000u) bad = true;
    }
#pragma unroll
    for (int j = 0; j < UN; ++j) {
      const uint32_t key = keys[j];
      bool in = valid[j] && (key & hi_mask) == prefix;
      uint32_t d = (key >> shift) & (nb - 1u);
      // plain shared-memory atomics: measured three times faster than aggregating equal digits within the warp first
      // (match.any + ballot per entry), although gradients crowd into a few exponent bins
      if (in) atomicAdd(&sh[d], 1u);
    }
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < nb; i += blockDim.x) {
    uint32_t c = sh[i];
    if (c) atomicAdd(&hist[i], c);
  }
  if (bad) atomicOr(flags, 2);
}

// Walk the histogram from the largest digit down until the cumulative count
// reaches the wanted rank; fix that digit in the prefix.
__global__ void __launch_bounds__(1024) sel_pick_kernel(const uint32_t* __restrict__ hist, int pass, SelState* st) {
  __shared__ uint32_t sc[kSelMaxBins];
  __shared__ uint32_t wsum[32];
  const int bits = sel_bits(pass), shift = sel_shift(pass);
  const int nb = 1 << bits;
  const int t = threadIdx.x;
  // reversed order: position p <-> digit nb-1-p; two consecutive positions per thread
  uint32_t a0 = (2 * t < nb) ? hist[nb - 1 - 2 * t] : 0u;
  uint32_t a1 = (2 * t + 1 < nb) ? hist[nb - 2 - 2 * t] : 0u;
  uint32_t s = a0 + a1, incl = s;
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
    if ((t & 31) >= o) incl += v;
  }
  if ((t & 31) == 31) wsum[t >> 5] = incl;
  __syncthreads();
  if (t < 32) {
    uint32_t w = wsum[t], wi = w;
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t v = __shfl_up_sync(0xffffffffu, wi, o);
      if (t >= o) wi += v;
    }
    wsum[t] = wi - w;   // exclusive
  }
  __syncthreads();
  uint32_t excl = wsum[t >> 5] + incl - s;
  if (2 * t < nb) sc[2 * t] = excl + a0;            // inclusive cumulative counts, descending digits
  if (2 * t + 1 < nb) sc[2 * t + 1] = excl + a0 + a1;
  __syncthreads();
  const uint32_t krem = st->krem;
  __syncthreads();   // everyone has read krem before the one matching thread rewrites it
  for (int p = t; p < nb; p += blockDim.x) {
    uint32_t cur = sc[p], prev = p ? sc[p - 1] : 0u;
    if (prev < krem && krem <= cur) {               // exactly one p satisfies this when krem >= 1
      uint32_t d = (uint32_t)(nb - 1 - p);
      uint32_t np = st->prefix | (d << shift);
      st->prefix = np;
      st->krem = krem - prev;
      if (pass == 2) { st->thr = np; st->take_eq = krem - prev; }
      if (pass == 0) st->use_cand = (cur - prev <= st->cand_cap) ? 1u : 0u;      // cur - prev: keys in the bucket
    }
  }
}

// Per block of kChunk consecutive entries: how many keys lie above / at the threshold.
template <class S, bool TOPK>
__global__ void __launch_bounds__(kChunkThreads) sel_count_kernel(const void* __restrict__ g, uint32_t n,
                                                                  const SelState* __restrict__ st,
                                                                  uint32_t* __restrict__ blk_gt,
                                                                  uint32_t* __restrict__ blk_eq, SelKey kp) {
  __shared__ uint32_t sg[kChunkThreads / 32], se[kChunkThreads / 32];
  if (st->use_cand) return;                    // counted from the candidate buffer instead
  const uint32_t thr = st->thr;
  const uint32_t nblk = (n + kChunk - 1) / kChunk;
  // a block walks over blocks of kChunk entries (the grid is a few blocks per SM, so that the launch costs little
  // when the kernel has nothing to do)
  for (uint32_t blk = blockIdx.x; blk < nblk; blk += gridDim.x) {
    const uint32_t base = blk * (uint32_t)kChunk;
    uint32_t cg = 0, ce = 0;
    // coalesced order here: only totals matter
    for (int r = 0; r < kChunk / kChunkThreads; ++r) {
      uint32_t i = base + r * kChunkThreads + threadIdx.x;
      if (i < n) {
        uint32_t key = TOPK ? mag_key(S::load(g, i)) : sel_key(S::load(g, i), i, kp);
        cg += key > thr; ce += key == thr;
      }
    }
    for (int o = 16; o; o >>= 1) { cg += __shfl_xor_sync(0xffffffffu, cg, o); ce += __shfl_xor_sync(0xffffffffu, ce, o); }
    if ((threadIdx.x & 31) == 0) { sg[threadIdx.x >> 5] = cg; se[threadIdx.x >> 5] = ce; }
    __syncthreads();
    if (threadIdx.x == 0) {
      uint32_t a = 0, b = 0;
      for (int w = 0; w < kChunkThreads / 32; ++w) { a += sg[w]; b += se[w]; }
      blk_gt[blk] = a; blk_eq[blk] = b;
    }
    __syncthreads();
  }
}

// The pass that copies the threshold bucket: per block of kChunk entries, the keys whose first digit is the chosen
// one go to a run of the candidate buffer (the block reserves it with one atomic add: where a run lies depends on the
// order the blocks arrive in, what it holds does not, and nothing downstream looks at more than the multiset of keys of
// a run), and the keys with a larger first digit are counted.
template <class S, bool TOPK>
__global__ void __launch_bounds__(kChunkThreads) sel_gather_kernel(const void* __restrict__ g, uint32_t n, SelState* st,
                                                                   uint32_t* __restrict__ blk_gt, uint32_t* __restrict__ blk_eq,
                                                                   uint32_t* __restrict__ cand, uint32_t* __restrict__ cand_start,
                                                                   uint32_t* __restrict__ cand_cnt, SelKey kp) {
  __shared__ uint32_t sg[kChunkThreads / 32], sc[kChunkThreads / 32], run_base;
  if (!st->use_cand) return;
  constexpr int EPT = kChunk / kChunkThreads;
  const uint32_t d0 = st->prefix >> sel_shift(0);
  const uint32_t base = blockIdx.x * (uint32_t)kChunk;
  const int t = threadIdx.x;
  uint32_t mine[EPT];
  uint32_t cg = 0, cc = 0;
#pragma unroll
  for (int r = 0; r < EPT; ++r) {
    const uint32_t i = base + r * kChunkThreads + t;
    uint32_t key = 0u; bool in = false;
    if (i < n) {
      key = TOPK ? mag_key(S::load(g, i)) : sel_key(S::load(g, i), i, kp);
      const uint32_t d = key >> sel_shift(0);
      cg += d > d0; in = d == d0;
    }
    mine[r] = key;
    cc |= in ? (1u << r) : 0u;               // which of this thread's entries are candidates
  }
  const uint32_t nc = __popc(cc);
  uint32_t ig = cg, ic = nc;
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t vg = __shfl_up_sync(0xffffffffu, ig, o), vc = __shfl_up_sync(0xffffffffu, ic, o);
    if ((t & 31) >= o) { ig += vg; ic += vc; }
  }
  if ((t & 31) == 31) { sg[t >> 5] = ig; sc[t >> 5] = ic; }
  __syncthreads();
  uint32_t woff = 0, tot_g = 0, tot_c = 0;
  for (int w = 0; w < kChunkThreads / 32; ++w) { if (w < (t >> 5)) woff += sc[w]; tot_g += sg[w]; tot_c += sc[w]; }
  if (t == 0) {
    run_base = tot_c ? atomicAdd(&st->cand_total, tot_c) : 0u;
    blk_gt[blockIdx.x] = tot_g; blk_eq[blockIdx.x] = 0u;
  }
  __syncthreads();
  const uint32_t rb = run_base;
  if (t == 0) { cand_start[blockIdx.x] = rb; cand_cnt[blockIdx.x] = tot_c; }
  uint32_t pos = rb + woff + ic - nc;
#pragma unroll
  for (int r = 0; r < EPT; ++r)
    if (cc & (1u << r)) cand[pos++] = mine[r];
}

// Histogram of the current digit over the candidate keys whose higher bits equal the prefix chosen so far.
__global__ void __launch_bounds__(512) sel_hist_keys_kernel(const uint32_t* __restrict__ cand, int pass,
                                                           const SelState* __restrict__ st, uint32_t* __restrict__ hist) {
  __shared__ uint32_t sh[kSelMaxBins];
  if (!st->use_cand) return;
  const int bits = sel_bits(pass), shift = sel_shift(pass);
  const uint32_t nb = 1u << bits, n = st->cand_total;
  for (uint32_t i = threadIdx.x; i < nb; i += blockDim.x) sh[i] = 0u;
  __syncthreads();
  const uint32_t prefix = st->prefix;
  const uint32_t hi_mask = 0xffffffffu << (shift + bits);
  const uint32_t stride = gridDim.x * blockDim.x;
  for (uint32_t b0 = blockIdx.x * blockDim.x; b0 < n; b0 += stride) {
    const uint32_t i = b0 + threadIdx.x;
    const uint32_t key = i < n ? cand[i] : 0u;
    const bool in = i < n && (key & hi_mask) == prefix;
    const uint32_t d = (key >> shift) & (nb - 1u);
    if (in) atomicAdd(&sh[d], 1u);
  }
  __syncthreads();
  for (uint32_t i = threadIdx.x; i < nb; i += blockDim.x) {
    const uint32_t c = sh[i];
    if (c) atomicAdd(&hist[i], c);
  }
}

// Per block of kChunk entries: the keys above / at the final threshold = those above the bucket (counted by the
// copying pass) + those of the block's run of candidates above / at it.  One thread per block.
__global__ void __launch_bounds__(256) sel_count_cand_kernel(const uint32_t* __restrict__ cand,
                                                            const uint32_t* __restrict__ cand_start,
                                                            const uint32_t* __restrict__ cand_cnt,
                                                            const SelState* __restrict__ st, uint32_t* __restrict__ blk_gt,
                                                            uint32_t* __restrict__ blk_eq, uint32_t nblk) {
  if (!st->use_cand) return;
  const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= nblk) return;
  const uint32_t thr = st->thr, s0 = cand_start[b], c = cand_cnt[b];
  uint32_t cg = 0, ce = 0;
  for (uint32_t j = 0; j < c; ++j) { const uint32_t key = cand[s0 + j]; cg += key > thr; ce += key == thr; }
  blk_gt[b] += cg; blk_eq[b] = ce;
}

// In-place exclusive scan of the per-block counts (single block; eight consecutive counts per thread and round).
__global__ void __launch_bounds__(1024) sel_scan_kernel(uint32_t* __restrict__ blk_gt, uint32_t* __restrict__ blk_eq,
                                                       uint32_t nblk) {
  constexpr int PT = 8;
  __shared__ uint32_t wg[32], we[32];
  __shared__ uint32_t carry_g, carry_e;
  const int t = threadIdx.x;
  if (t == 0) { carry_g = 0; carry_e = 0; }
  __syncthreads();
  for (uint32_t base = 0; base < nblk; base += 1024 * PT) {
    const uint32_t i0 = base + (uint32_t)t * PT;
    uint32_t vg[PT], ve[PT], g = 0, e = 0;
#pragma unroll
    for (int j = 0; j < PT; ++j) {
      vg[j] = (i0 + j < nblk) ? blk_gt[i0 + j] : 0u; ve[j] = (i0 + j < nblk) ? blk_eq[i0 + j] : 0u;
      g += vg[j]; e += ve[j];
    }
    uint32_t ig = g, ie = e;
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t ug = __shfl_up_sync(0xffffffffu, ig, o), ue = __shfl_up_sync(0xffffffffu, ie, o);
      if ((t & 31) >= o) { ig += ug; ie += ue; }
    }
    if ((t & 31) == 31) { wg[t >> 5] = ig; we[t >> 5] = ie; }
    __syncthreads();
    if (t < 32) {
      uint32_t a = wg[t], b = we[t], ia = a, ib = b;
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t va = __shfl_up_sync(0xffffffffu, ia, o), vb = __shfl_up_sync(0xffffffffu, ib, o);
        if (t >= o) { ia += va; ib += vb; }
      }
      wg[t] = ia - a; we[t] = ib - b;
    }
    __syncthreads();
    uint32_t xg = carry_g + wg[t >> 5] + ig - g, xe = carry_e + we[t >> 5] + ie - e;    // exclusive prefix of this thread's run
#pragma unroll
    for (int j = 0; j < PT; ++j) {
      if (i0 + j < nblk) { blk_gt[i0 + j] = xg; blk_eq[i0 + j] = xe; }
      xg += vg[j]; xe += ve[j];
    }
    __syncthreads();
    if (t == 1023) { carry_g = xg; carry_e = xe; }
    __syncthreads();
  }
}

// Ordered compaction: entry i belongs to Omega iff key > thr, or key == thr and
// fewer than take_eq equal keys precede it.  Its slot is the number of selected
// entries before it, so Omega comes out strictly ascending.  The selected values
// are saved to g_s (fp32 complex) for the residual/restore passes of the refresh.
template <class S, bool TOPK>
__global__ void __launch_bounds__(kChunkThreads) sel_compact_kernel(const void* __restrict__ g, uint32_t n,
                                                                    const SelState* __restrict__ st,
                                                                    const uint32_t* __restrict__ blk_gt,
                                                                    const uint32_t* __restrict__ blk_eq,
                                                                    uint32_t* __restrict__ omega,
                                                                    cf* __restrict__ g_s, uint32_t k, SelKey kp) {
  __shared__ uint32_t wsum[kChunkThreads / 32];
  constexpr int EPT = kChunk / kChunkThreads;   // 8 consecutive entries per thread
  const uint32_t thr = st->thr, take = st->take_eq;
  const uint32_t base = blockIdx.x * (uint32_t)kChunk + threadIdx.x * EPT;
  cf v[EPT];
  uint32_t key[EPT];
  uint32_t cnt = 0;   // packed: eq count in the high half, gt count in the low half
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    uint32_t i = base + e;
    if (i < n) { v[e] = S::load(g, i); key[e] = TOPK ? mag_key(v[e]) : sel_key(v[e], i, kp); } else { v[e] = make_float2(0.f, 0.f); key[e] = 0u; }
    bool valid = i < n;
    cnt += (valid && key[e] > thr) ? 1u : 0u;
    cnt += (valid && key[e] == thr) ? 0x10000u : 0u;
  }
  uint32_t incl = cnt;
  const int t = threadIdx.x;
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t u = __shfl_up_sync(0xffffffffu, incl, o);
    if ((t & 31) >= o) incl += u;
  }
  if ((t & 31) == 31) wsum[t >> 5] = incl;
  __syncthreads();
  uint32_t woff = 0;
  for (int w = 0; w < (t >> 5); ++w) woff += wsum[w];
  uint32_t excl = woff + incl - cnt;
  uint32_t gt_before = blk_gt[blockIdx.x] + (excl & 0xffffu);
  uint32_t eq_before = blk_eq[blockIdx.x] + (excl >> 16);
#pragma unroll
  for (int e = 0; e < EPT; ++e) {
    uint32_t i = base + e;
    if (i >= n) break;
    bool isgt = key[e] > thr, iseq = key[e] == thr;
    bool sel = isgt || (iseq && eq_before < take);
    if (sel) {
      uint32_t pos = gt_before + (eq_before < take ? eq_before : take);
      if (pos < k) { omega[pos] = i; g_s[pos] = v[e]; }
    }
    gt_before += isgt; eq_before += iseq;
  }
}

// R = G - Sparse(G, Omega): zero the entries at Omega in place ...
template <class S>
__global__ void scatter_zero_kernel(void* __restrict__ g, const uint32_t* __restrict__ omega, uint32_t k) {
  uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < k) S::store(g, omega[j], make_float2(0.f, 0.f));
}
// ... and put the saved values back once the factor matrices are computed.
template <class S>
__global__ void scatter_restore_kernel(void* __restrict__ g, const uint32_t* __restrict__ omega,
                                       const cf* __restrict__ g_s, uint32_t k) {
  uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < k) S::store(g, omega[j], g_s[j]);
}

// slab_ptr[s] = number of Omega entries below s*E (s = 0..nslab): the ascending index list is
// thereby grouped by slab, and the streaming kernels find their slab's entries with two loads.
__global__ void slab_ptr_kernel(const uint32_t* __restrict__ omega, uint32_t k, uint32_t E, uint32_t nslab,
                                uint32_t* __restrict__ slab_ptr) {
  uint32_t s = blockIdx.x * blockDim.x + threadIdx.x;
  if (s > nslab) return;
  uint64_t key = (uint64_t)s * E;
  slab_ptr[s] = (s == nslab) ? k : (uint32_t)lower_bound_u32(omega, (int)k, (uint32_t)key);
}

}  // namespace tg
