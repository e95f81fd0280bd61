// Mode-n Gram matrices A_n = R_(n) R_(n)^H (TuckerFactors of Algorithm 1: the factor matrices are the leading
// eigenvectors of A_n) on the 5th-generation tensor cores, for the modes whose rows are long contiguous runs:
// the tensor seen as [O][I_n][C] with C contiguous, C * entry size a multiple of 16 bytes and 64 <= I_n <= 256.
//
// With a row as the interleaved real vector x_a = (re, im, re, im, ...) of length 2C,
//   Re A[a][b] = x_a . x_b,    Im A[a][b] = x_a . y_b,    y_b = (-im, re, -im, re, ...),
// i.e. one real product D = X [X; Y]^T with K = 2 O C.  The contraction range is cut into tiles of 128 bytes per
// row; a stage of the ring holds 1, 2 or 4 of them (more for fewer rows).  Per piece:
//   * one thread issues a tiled TMA load of the I_n x 128-byte box (128-byte swizzle, rows beyond I_n and bytes
//     beyond the run zero-filled) into the X half of a stage;
//   * four warps make the Y half from it, 16 bytes at a time at the same offset (the swizzle permutes 16-byte pieces
//     of a row, and a (re, im) pair never straddles one), and for fp32 storage round X in place to TF32 (the
//     tensor core would truncate);
//   * one thread issues tcgen05.mma (M = 128 rows of X from shared memory as the A operand, B = X and Y, fp32
//     accumulators in tensor memory: Re in columns [0, I_n), Im in [256, 256 + I_n); when 2 I_n <= 256, one
//     instruction of N = 2 I_n with Im at column I_n) and commits the stage back to the loader.
// 16-bit storage is contracted exactly (kind::f16, fp16 or bfloat16 operands as stored, products exact in fp32).
// Grid = splits of the contraction range; a launch computes the first 128 rows of A for the rows it is given.  A
// matrix of more than 128 rows takes two launches: rows 0..127 against all columns (B = all rows, all 512 columns of
// tensor memory), then the same kernel on the rows from 128 on alone (A is Hermitian: their columns below 128 are
// the first launch's), which loads and multiplies half as much.  The tensor core adds into its fp32 accumulator with
// truncation, which biases a long chain (measured: 6e-5 of the diagonal after 676 instructions), so the chain is cut
// into groups of tiles: after each group four more warps move the accumulators out of tensor memory and add them,
// with ordinary fp32 adds, into the block's own partial[split][a][b] (entries on and above the diagonal's 16-column
// piece only), while the next group accumulates into the other half of tensor memory (I_n <= 128; larger I_n
// fill all 512 columns, and the tensor core waits for the drain).  The partials are summed in a fixed order by
// gram_reduce_kernel: every sum is formed in one order, so the result is deterministic.  Every wait is bounded; a
// wait that runs out sets the sticky copy-timeout flag, the block drains what it started, frees its tensor memory
// and returns.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "ptx.cuh"

namespace tg {

constexpr int GT_THREADS = 320;        // warp 0: TMA + tensor-memory owner, 1: MMA issue, 2-5: Y tiles, 6-9: accumulator drain
constexpr int GT_WORKERS = 128;
constexpr int GT_DRAINERS = 128;
constexpr int GT_ROW_BYTES = 128;
constexpr int GT_MIN_ROWS = 64;        // the A operand reads 128 rows of a stage: X and Y together must hold them
constexpr int GT_MAX_ROWS = 256;
constexpr int GT_TMEM_COLS = 512;
constexpr int GT_IM_COL = 256;
constexpr int GT_MAX_STAGES = 4;       // measured on 128 rows of fp32: 126 / 96 / 91 / 123 / 128 us with 2 / 3 / 4 / 5 / 6 stages
constexpr uint32_t GT_WAIT_LIMIT = 1u << 22;      // polls of a wait, and
constexpr uint64_t GT_WAIT_NS = 1000000000ull;     // its limit in nanoseconds of the global timer

struct GramTcParams {
  int In;                    // rows of this launch: rows row0 .. row0 + In of the unfolding
  int rows;                  // In rounded up to a multiple of 16: rows of a tile
  int row0;                  // first row
  int a_min;                 // rows of A below this one belong to another launch and are not written
  int ld;                    // rows (= columns) of the whole Gram matrix
  int stages;
  int kt;                    // 128-byte pieces of every row per stage (a tile)
  uint32_t tiles_per_o;      // tiles per run of C entries
  uint32_t tiles_total;      // O * tiles_per_o
  uint32_t tiles_per_split;
  uint32_t group_tiles;      // tiles accumulated in tensor memory before the sums move to the partial matrix
  cf* partial;               // [splits][ld][ld]
  int* flags;
};

constexpr size_t GT_STAGING = 4 * 32 * 128;     // per drain warp: 32 rows x 16 complex sums
inline size_t gram_tc_smem(int rows, int stages, int kt) { return (size_t)stages * kt * 2 * rows * GT_ROW_BYTES + GT_STAGING + 1024; }

// wait on an mbarrier phase; gives up when the limit runs out or another thread of the block has given up
__device__ __forceinline__ bool gt_wait(uint64_t* bar, uint32_t parity, volatile int* failed) {
  uint64_t start = 0;
  for (uint32_t i = 0; i < GT_WAIT_LIMIT; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63) == 63) {
      if (*failed) return false;
      uint64_t now;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
      if (start == 0) start = now;
      else if (now - start > GT_WAIT_NS) return false;
    }
  }
  return false;
}

// FMT: 0 fp16 pairs, 1 bfloat16 pairs, 2 fp32 pairs (contracted as TF32)
template <int FMT>
__global__ void __launch_bounds__(GT_THREADS, 1) gram_tc_kernel(const __grid_constant__ CUtensorMap tmap, const GramTcParams P) {
  extern __shared__ unsigned char gt_raw[];
  __shared__ __align__(8) uint64_t full[GT_MAX_STAGES], ready[GT_MAX_STAGES], empty[GT_MAX_STAGES], acc_full[2], acc_free[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int failed_s;
  volatile int* failed = &failed_s;
  constexpr bool TF32 = FMT == 2;
  constexpr int BOXK = TF32 ? 32 : 64;                  // elements of the tensor map per 128-byte row piece
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t raw = smem_u32(gt_raw);
  const uint32_t tiles0 = (raw + 1023u) & ~1023u;       // swizzled tiles sit on 1,024-byte boundaries
  unsigned char* tiles_p = gt_raw + (tiles0 - raw);
  // a stage: KT pieces, each the X half (rows x 128 bytes) followed by its Y half
  const int KT = P.kt;
  const uint32_t tile_bytes = (uint32_t)P.rows * GT_ROW_BYTES, piece_bytes = 2 * tile_bytes, stage_bytes = piece_bytes * (uint32_t)KT;
  const int stages = P.stages;
  const uint32_t t0 = blockIdx.x * P.tiles_per_split;
  const uint32_t t1 = min(t0 + P.tiles_per_split, P.tiles_total);
  const uint32_t n = t1 > t0 ? t1 - t0 : 0;
  const uint32_t F = P.group_tiles;
  const bool single = 2 * P.rows <= 256;                // Re and Im columns from one instruction, two accumulator sets
  const int im_col = single ? P.rows : GT_IM_COL;
  const uint32_t nbuf = single ? 2 : 1;

  if (tid == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], GT_WORKERS); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_free[b], GT_DRAINERS); }
    failed_s = 0;
    fence_mbar_init();
  }
  if (warp == 0) { tmem_alloc(&tmem_slot, GT_TMEM_COLS); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;

  if (warp == 0) {
    // ---- loader ----
    if (lane == 0) {
      uint32_t it = 0;
      for (; it < n; ++it) {
        const int s = it % stages; const uint32_t ph = (it / stages) & 1;
        if (!gt_wait(&empty[s], ph ^ 1, failed)) { atomicOr(P.flags, 4); *failed = 1; break; }
        mbar_expect_tx(&full[s], tile_bytes * (uint32_t)KT);
        const uint32_t t = t0 + it, o = t / P.tiles_per_o, kt = (t - o * P.tiles_per_o) * (uint32_t)KT;
        // (a piece beyond the end of the run starts outside the tensor and arrives as zeros)
        for (int j = 0; j < KT; ++j)
          tma_load_3d(tiles0 + s * stage_bytes + j * piece_bytes, &tmap, (int)((kt + j) * BOXK), P.row0, (int)o, &full[s]);
      }
      if (*failed) {
        // loads still in flight must land before the block's shared memory is given up
        for (uint32_t j = it > (uint32_t)stages ? it - stages : 0; j < it; ++j)
          mbar_wait_bounded(&full[j % stages], (j / stages) & 1, 1u << 16);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issue ----
    if (lane == 0) {
      const uint32_t idesc = umma_idesc(FMT, single ? 2 * P.rows : P.rows);
      uint32_t in_group = 0, g = 0;
      for (uint32_t it = 0; it < n; ++it) {
        const uint32_t b = g % nbuf;
        if (in_group == 0) {                             // the drain of this accumulator set's previous group is over
          if (!gt_wait(&acc_free[b], ((g / nbuf) & 1) ^ 1, failed)) { atomicOr(P.flags, 4); *failed = 1; break; }
        }
        const int s = it % stages; const uint32_t ph = (it / stages) & 1;
        if (!gt_wait(&ready[s], ph, failed)) { atomicOr(P.flags, 4); *failed = 1; break; }
        tc_fence_after_sync();
        const uint32_t d = tmem + b * 256u;
        for (int j = 0; j < KT; ++j) {
          const uint32_t xs = tiles0 + s * stage_bytes + j * piece_bytes;
          const uint64_t dx = umma_desc_k128(xs), dy = umma_desc_k128(xs + tile_bytes);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {               // 32 bytes of every row per instruction
            const bool acc = in_group != 0 || j != 0 || ks != 0;
            const uint64_t adv = (uint64_t)(ks * 32 >> 4);
            umma_ss<TF32>(d, dx + adv, dx + adv, idesc, acc);
            if (!single) umma_ss<TF32>(d + GT_IM_COL, dx + adv, dy + adv, idesc, acc);
          }
        }
        umma_commit(&empty[s]);
        if (++in_group == F || it + 1 == n) { umma_commit(&acc_full[b]); in_group = 0; ++g; }
      }
    }
    __syncwarp();
  } else if (warp < 6) {
    // ---- Y tiles ----
    const int w = tid - 64;
    const int nchunks = P.rows * (GT_ROW_BYTES / 16);
    for (uint32_t it = 0; it < n; ++it) {
      const int s = it % stages; const uint32_t ph = (it / stages) & 1;
      if (!gt_wait(&full[s], ph, failed)) { atomicOr(P.flags, 4); *failed = 1; break; }
      for (int pj = 0; pj < KT; ++pj) {
      uint4* x = reinterpret_cast<uint4*>(tiles_p + (size_t)s * stage_bytes + (size_t)pj * piece_bytes);
      uint4* y = reinterpret_cast<uint4*>(tiles_p + (size_t)s * stage_bytes + (size_t)pj * piece_bytes + tile_bytes);
      // eight 16-byte pieces per thread in flight: all loads of a batch before its first store (the stores may not
      // overtake loads the compiler cannot prove disjoint)
      for (int c = w; c < nchunks; c += 8 * GT_WORKERS) {
        uint4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c + j * GT_WORKERS < nchunks) v[j] = x[c + j * GT_WORKERS];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (c + j * GT_WORKERS >= nchunks) break;
          uint4 r = v[j], o;
          if (TF32) {
            r.x = (r.x + 0x1000u) & 0xffffe000u; r.y = (r.y + 0x1000u) & 0xffffe000u;
            r.z = (r.z + 0x1000u) & 0xffffe000u; r.w = (r.w + 0x1000u) & 0xffffe000u;
            x[c + j * GT_WORKERS] = r;
            o.x = r.y ^ 0x80000000u; o.y = r.x; o.z = r.w ^ 0x80000000u; o.w = r.z;
          } else {
            // word = re | im << 16  ->  (-im) | re << 16
            o.x = ((r.x >> 16) ^ 0x8000u) | (r.x << 16); o.y = ((r.y >> 16) ^ 0x8000u) | (r.y << 16);
            o.z = ((r.z >> 16) ^ 0x8000u) | (r.z << 16); o.w = ((r.w >> 16) ^ 0x8000u) | (r.w << 16);
          }
          y[c + j * GT_WORKERS] = o;
        }
      }
      }
      fence_async_smem();
      mbar_arrive(&ready[s]);
    }
  } else {
    // ---- drain: tensor memory -> partial[split][a][b], one group of tiles at a time ----
    const int q = warp & 3;                              // the 32 lanes of tensor memory this warp may read
    const int a = q * 32 + lane;                         // row of the tile; row0 + a of the Gram matrix
    cf* out = P.partial + (size_t)blockIdx.x * P.ld * P.ld + (size_t)(P.row0 + a) * P.ld + P.row0;
    const int c_first = (q * 32) & ~15;                  // pieces left of the diagonal are not needed
    const uint32_t ngroups = (n + F - 1) / F;
    const bool even = ((P.ld | P.row0) & 1) == 0;        // the 16-column pieces start on 16-byte boundaries
    float4* stg = reinterpret_cast<float4*>(tiles_p + (size_t)stages * stage_bytes) + (warp - 6) * 256;
    for (uint32_t g = 0; g < ngroups; ++g) {
      const uint32_t b = g % nbuf;
      bool ok = gt_wait(&acc_full[b], (g / nbuf) & 1, failed);
      if (!ok && !*failed) { atomicOr(P.flags, 4); *failed = 1; }
      ok = __all_sync(0xffffffffu, ok);                  // the tensor-memory loads below are warp-wide
      if (!ok) break;
      tc_fence_after_sync();
      const uint32_t ta0 = tmem + b * 256u + ((uint32_t)(q * 32) << 16);
      for (int c0 = c_first; c0 < P.rows; c0 += 16) {
        uint32_t re[16], im[16];
        tmem_ld16(ta0 + (uint32_t)c0, re);
        tmem_ld16(ta0 + (uint32_t)(im_col + c0), im);
        tmem_wait_ld();
        if (even) {
          // through shared memory, so that a warp touches whole 128-byte rows of the partial matrix: lane = row on
          // the way in (16-byte units rotated by the row, conflict-free), 8 lanes per row on the way out
#pragma unroll
          for (int u = 0; u < 8; ++u)
            stg[lane * 8 + (u ^ (lane & 7))] = make_float4(__uint_as_float(re[2 * u]), __uint_as_float(im[2 * u]),
                                                           __uint_as_float(re[2 * u + 1]), __uint_as_float(im[2 * u + 1]));
          __syncwarp();
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int row = 4 * i + (lane >> 3), u = lane & 7;
            float4 v = stg[row * 8 + (u ^ (row & 7))];
            const int ar = a - lane + row;
            if (ar < P.In && P.row0 + ar >= P.a_min && c0 + 2 * u < P.In) {
              float4* dst = reinterpret_cast<float4*>(out + (ptrdiff_t)(row - lane) * P.ld + c0) + u;
              if (g != 0) { const float4 w = *dst; v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w; }
              *dst = v;
            }
          }
          __syncwarp();
        } else if (a < P.In && P.row0 + a >= P.a_min) {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (c0 + j < P.In) {
              cf v = make_float2(__uint_as_float(re[j]), __uint_as_float(im[j]));
              if (g != 0) { const cf u = out[c0 + j]; v.x += u.x; v.y += u.y; }
              out[c0 + j] = v;
            }
        }
      }
      tc_fence_before_sync();
      mbar_arrive(&acc_free[b]);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, GT_TMEM_COLS);
}

}  // namespace tg
