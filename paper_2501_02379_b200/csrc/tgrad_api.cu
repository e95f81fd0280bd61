// Host side of the C ABI: state layout, argument checks, stage scheduling on the
// caller's stream.  Every step of the path runs in the kernels of this library;
// there is no CPU or library fallback.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/tgrad.h"
#include "common.cuh"
#include "gram.cuh"
#include "gram_tc.cuh"
#include "jacobi.cuh"
#include "modeprod.cuh"
#include "select.cuh"
#include "subspace.cuh"
#include "tail.cuh"
#include "tail_tc.cuh"
#include "tail_h.cuh"

using namespace tg;

namespace {

std::atomic<int64_t> g_launches{0};

constexpr int kStages = 5;   // proj_tail, proj_chain, adam_core, back_chain, back_tail
constexpr int kTimingRing = 64;

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }
constexpr size_t kSmemMax = 227 * 1024;   // dynamic shared memory a block may ask for

struct Layout {
  // persistent block
  size_t p_flags, p_omega, p_slab, p_factor[TGRAD_MAX_NDIM], p_ml, p_vl, p_ms, p_vs, p_u2tab, p_total;
  uint32_t nslab, E;          // slabs of the trailing two modes, entries per slab
  // workspace block
  size_t w_ns, w_gs, w_core, w_nl, w_bufa, w_bufb, w_sel, w_hist, w_blk, w_gram[TGRAD_MAX_NDIM], w_jac[TGRAD_MAX_NDIM],
      w_v[TGRAD_MAX_NDIM], w_log[TGRAD_MAX_NDIM], w_lam[TGRAD_MAX_NDIM], w_partial, w_hooi0, w_hooi1, w_ident, w_rbuf, w_diag, w_total;
  uint32_t hooi_smem;         // shared memory of the compression kernel when one trailing factor is replaced by the identity
  bool jac_fast[TGRAD_MAX_NDIM];    // eigensolver with the matrix in shared memory and a rotation log
  uint64_t numel, P, tsize;   // entries, core entries, entries of the tail-contracted tensor
  uint32_t nblk;              // compaction blocks
  int gram_splits[TGRAD_MAX_NDIM];
  uint32_t gram_chunks[TGRAD_MAX_NDIM], gram_cps[TGRAD_MAX_NDIM];
};

struct TailPlan {
  // general path: one block per slab
  TailBlkGeom bproj, bback;
  uint32_t hooi_smem;      // shared memory of the compression kernel in a refinement sweep (0: no refinement)
  int grid_bproj, grid_bback;
  // tensor-core fast path (complex64 storage, 16/32/64 slab rows, small trailing ranks)
  bool tc;
  int rat, ks, ntw, pjw, back_ns;
  TcGeom gproj, gback;
  int grid_proj, grid_back;
  // half-storage compression kernel (fp16 MMA)
  bool th, thb;
  int h_rat, h_rbt, grid_h, grid_hb;
  TailHGeom gh;
  TailHBGeom ghb;
};

tgrad_status validate(const tgrad_config* c) {
  if (!c) return TGRAD_ERR_INVALID_ARG;
  if (c->ndim < 2 || c->ndim > TGRAD_MAX_NDIM) return TGRAD_ERR_INVALID_ARG;
  long double tot = 1;
  for (int n = 0; n < c->ndim; ++n) {
    if (c->dims[n] < 1) return TGRAD_ERR_INVALID_ARG;
    if (c->ranks[n] < 1 || c->ranks[n] > c->dims[n]) return TGRAD_ERR_INVALID_ARG;
    tot *= (long double)c->dims[n];
  }
  if (c->k < 0 || (long double)c->k > tot) return TGRAD_ERR_INVALID_ARG;
  if (c->T < 1) return TGRAD_ERR_INVALID_ARG;
  if (c->wg_dtype != TGRAD_C64 && c->wg_dtype != TGRAD_C32H && c->wg_dtype != TGRAD_C32B) return TGRAD_ERR_INVALID_ARG;
  if (!(c->beta1 >= 0.f && c->beta1 < 1.f) || !(c->beta2 >= 0.f && c->beta2 < 1.f) || !(c->eps >= 0.f))
    return TGRAD_ERR_INVALID_ARG;
  if (c->jacobi_max_sweeps < 0 || c->jacobi_tol < 0.f) return TGRAD_ERR_INVALID_ARG;
  if (c->warm_refresh != 0 && c->warm_refresh != 1) return TGRAD_ERR_INVALID_ARG;
  if (c->hooi_iters < 0 || c->hooi_iters > 64) return TGRAD_ERR_INVALID_ARG;
  if (c->composition < 0 || c->composition > 2 || c->sparse_strategy < 0 || c->sparse_strategy > 2) return TGRAD_ERR_INVALID_ARG;
  // limits of this implementation
  if (tot >= 4294967296.0L) return TGRAD_ERR_UNSUPPORTED;    // flat indices are uint32
  if (c->k >= ((int64_t)1 << 31)) return TGRAD_ERR_UNSUPPORTED;   // slots of Omega are addressed with int
  for (int n = 0; n < c->ndim; ++n)
    if (c->dims[n] > JAC_MAX_N) return TGRAD_ERR_UNSUPPORTED;
  if (c->ranks[c->ndim - 1] > 32) return TGRAD_ERR_UNSUPPORTED;
  return TGRAD_OK;
}


// Split-K plan of one Gram accumulation: In x In output, contraction over O * C entries per row.
void plan_gram_dims(int In, uint64_t O, uint64_t C, int sm, uint32_t& chunks, uint32_t& cps, int& splits) {
  uint64_t total = (O * C + GR_KT - 1) / GR_KT;      // the contraction index (o, c) is flattened
  int T = (In + GR_T - 1) / GR_T;
  int tiles = T * (T + 1) / 2;
  uint64_t want = (uint64_t)(6 * sm + tiles - 1) / tiles;
  if (want < 1) want = 1;
  if (want > 1024) want = 1024;
  if (want > total) want = total;
  if (want < 1) want = 1;
  uint64_t per = (total + want - 1) / want;
  if (per < 1) per = 1;
  chunks = (uint32_t)total; cps = (uint32_t)per; splits = (int)((total + per - 1) / per);
  if (splits < 1) splits = 1;
}
void plan_gram(const tgrad_config* c, int n, int sm, uint32_t& chunks, uint32_t& cps, int& splits) {
  uint64_t O = 1, C = 1;
  for (int m = 0; m < n; ++m) O *= c->dims[m];
  for (int m = n + 1; m < c->ndim; ++m) C *= c->dims[m];
  plan_gram_dims((int)c->dims[n], O, C, sm, chunks, cps, splits);
}

// Plan of the tcgen05 Gram kernel for a tensor seen as [O][In][C] with entries of `ebytes` bytes; ok = false when the
// shape does not suit it (rows that are not 16-byte multiples or too short for 128-byte tiles, a short contraction
// that wants the split-precision products, fewer than 64 or more than 256 rows) and the mma.sync kernel runs instead.
struct GramTcLaunch { int In, rows, row0, a_min, stages, kt; uint32_t tiles_per_o, tiles_total, per; int splits; };
struct GramTcPlan { bool ok; int nlaunch, splits; GramTcLaunch l[2]; };
constexpr int kGramTcMaxBlocks = 148;     // upper bound of the splits, whatever the device: sizes the scratch
GramTcPlan plan_gram_tc(int In, uint64_t O, uint64_t C, int ebytes, int sm) {
  GramTcPlan pl; memset(&pl, 0, sizeof(pl));
  const uint64_t run = C * (uint64_t)ebytes;           // bytes of one row's contiguous run
  if (In < GT_MIN_ROWS || In > GT_MAX_ROWS || run % 16 != 0 || run < 512 || O * C < 16384) return pl;
  const uint64_t per_o = (run + GT_ROW_BYTES - 1) / GT_ROW_BYTES, total = O * per_o;
  if (O >= (1ull << 31) || 2 * C >= (1ull << 32) || total >= (1ull << 32) || (uint64_t)In * run >= (1ull << 40)) return pl;
  const int rows = (In + 15) / 16 * 16;
  pl.nlaunch = rows > 128 ? 2 : 1;
  pl.l[0].In = In; pl.l[0].rows = rows; pl.l[0].row0 = 0; pl.l[0].a_min = 0;
  if (pl.nlaunch == 2) {
    // the rows from 128 on; at least 64 of them, so that the A operand's 128 rows stay inside a stage
    int row0 = 128;
    if (In - row0 < GT_MIN_ROWS) row0 = (In - GT_MIN_ROWS) & ~1;
    pl.l[1].In = In - row0; pl.l[1].rows = (In - row0 + 15) / 16 * 16; pl.l[1].row0 = row0; pl.l[1].a_min = 128;
  }
  if (sm > kGramTcMaxBlocks) sm = kGramTcMaxBlocks;
  for (int i = 0; i < pl.nlaunch; ++i) {
    GramTcLaunch& l = pl.l[i];
    // Pieces of 128 bytes per stage and stages, as measured (us per Gram matrix with pieces x stages = 1x4, 2x3, 4x3:
    // 64 rows of fp32 343 / 244 / 195, 96 rows of fp16 135 / 103 / -, 128 rows of fp32 99 / 123 / -): handing a
    // stage on costs about the same whatever its size, but more than about 96 KB of tiles in flight is slower again.
    const size_t piece = (size_t)2 * l.rows * GT_ROW_BYTES;
    int kt = l.rows <= 64 ? 4 : (l.rows < 128 ? 2 : 1);
    if ((uint64_t)kt > per_o) kt = (int)per_o;
    l.kt = kt;
    int st = (kt == 1 && l.rows <= 128) ? 4 : 3;
    const int fit = (int)((size_t)(200 << 10) / (piece * kt));
    if (st > fit) st = fit;
    if (st > GT_MAX_STAGES) st = GT_MAX_STAGES;
    if (st < 1) return pl;
    l.stages = st;
    const uint64_t tpo = (per_o + kt - 1) / kt, tot = O * tpo;
    uint64_t want = (uint64_t)(sm < 1 ? 1 : sm);
    if (want > tot) want = tot;
    const uint64_t per = (tot + want - 1) / want;
    l.tiles_per_o = (uint32_t)tpo; l.tiles_total = (uint32_t)tot; l.per = (uint32_t)per;
    l.splits = (int)((tot + per - 1) / per);
  }
  // both launches must write the same number of partial matrices (the reduction sums that many for every entry)
  if (pl.nlaunch == 2 && pl.l[0].splits != pl.l[1].splits) {
    const int common = pl.l[0].splits < pl.l[1].splits ? pl.l[0].splits : pl.l[1].splits;
    for (int i = 0; i < 2; ++i) {
      GramTcLaunch& l = pl.l[i];
      const uint64_t per = ((uint64_t)l.tiles_total + common - 1) / common;
      l.per = (uint32_t)per; l.splits = (int)(((uint64_t)l.tiles_total + per - 1) / per);
    }
    if (pl.l[0].splits != pl.l[1].splits) return pl;      // (short contractions only) leave it to the other kernel
  }
  pl.splits = pl.l[0].splits;
  pl.ok = true;
  return pl;
}

// The configuration the kernels see.  A matrix (N = 2, where the Tucker decomposition is the matrix SVD) is handled as
// the 3-way tensor I_1 x 1 x I_2 with ranks (r_1, 1, r_2): the unit mode's factor is the 1 x 1 identity, so every
// stage computes exactly what Algorithm 1 computes for the matrix.  map[n] = internal mode of the caller's mode n.
tgrad_status internal_config(const tgrad_config* ext, tgrad_config& in, int* map) {
  tgrad_status s = validate(ext);
  if (s != TGRAD_OK) return s;
  in = *ext;
  for (int n = 0; n < TGRAD_MAX_NDIM; ++n) map[n] = n;
  if (ext->ndim == 2) {
    in.ndim = 3;
    in.dims[0] = ext->dims[0]; in.dims[1] = 1; in.dims[2] = ext->dims[1];
    in.ranks[0] = ext->ranks[0]; in.ranks[1] = 1; in.ranks[2] = ext->ranks[1];
    map[0] = 0; map[1] = 2;
  }
  return TGRAD_OK;
}

tgrad_status compute_layout(const tgrad_config* c, Layout& L, int sm) {
  const int N = c->ndim;
  {
    // a trailing slab and the operand tables of its two products must fit in the shared memory of one SM
    const int A = (int)c->dims[N - 2], B = (int)c->dims[N - 1], ra = c->ranks[N - 2], rb = c->ranks[N - 1];
    if (tail_blk_geom(A, B, ra, rb, false).total > kSmemMax || tail_blk_geom(A, B, ra, rb, true).total > kSmemMax)
      return TGRAD_ERR_UNSUPPORTED;
  }
  uint64_t numel = 1, P = 1;
  for (int n = 0; n < N; ++n) { numel *= (uint64_t)c->dims[n]; P *= (uint64_t)c->ranks[n]; }
  L.numel = numel; L.P = P;
  uint64_t S = numel / ((uint64_t)c->dims[N - 1] * c->dims[N - 2]);
  L.tsize = S * c->ranks[N - 1] * c->ranks[N - 2];
  const uint64_t k = (uint64_t)c->k;
  size_t o = 0;
  L.p_flags = o; o = align_up(o + 64 * sizeof(int));
  L.p_omega = o; o = align_up(o + k * 4);
  L.nslab = (uint32_t)S; L.E = (uint32_t)((uint64_t)c->dims[N - 1] * c->dims[N - 2]);
  L.p_slab = o; o = align_up(o + ((size_t)S + 1) * 4);
  for (int n = 0; n < N; ++n) { L.p_factor[n] = o; o = align_up(o + (size_t)c->dims[n] * c->ranks[n] * 8); }
  L.p_ml = o; o = align_up(o + P * 8);
  L.p_vl = o; o = align_up(o + P * 4);
  L.p_ms = o; o = align_up(o + k * 8);
  L.p_vs = o; o = align_up(o + k * 4);
  // operand-fragment table of the compression kernel: 32 lanes x 32 bytes per (8-row tile, 8-column tile) of U^(N-1)
  L.p_u2tab = o; o = align_up(o + (size_t)((c->dims[N - 2] + 7) / 8) * ((c->ranks[N - 2] + 7) / 8) * 1024);
  L.p_total = o;
  o = 0;
  L.w_ns = o; o = align_up(o + k * 8);
  L.w_gs = o; o = align_up(o + k * 8);
  L.w_core = o; o = align_up(o + P * 8);
  L.w_nl = o; o = align_up(o + P * 8);
  L.w_bufa = o; o = align_up(o + L.tsize * 8);
  L.w_bufb = o; o = align_up(o + L.tsize * 8);
  L.w_sel = o; o = align_up(o + sizeof(SelState));
  L.w_hist = o; o = align_up(o + 3 * kSelMaxBins * 4);
  L.nblk = (uint32_t)((numel + kChunk - 1) / kChunk);
  L.w_blk = o; o = align_up(o + (size_t)4 * L.nblk * 4);      // per block: keys above / at the threshold, start and length of its run of candidates
  size_t partial = 0;
  for (int n = 0; n < N; ++n) {
    size_t sq = (size_t)c->dims[n] * c->dims[n] * 8;
    L.w_gram[n] = o; o = align_up(o + sq);   // A_n, kept for inspection
    L.w_jac[n] = o; o = align_up(o + (size_t)c->dims[n] * (c->dims[n] | 1) * 8);    // working copy the solver diagonalises
    L.w_v[n] = o; o = align_up(o + sq);      // accumulated rotations; scratch of the subspace iteration
    const int sweeps = c->jacobi_max_sweeps > 0 ? c->jacobi_max_sweeps : 30;
    const size_t logb = jac_log_entries((int)c->dims[n], sweeps) * sizeof(float4);
    L.jac_fast[n] = c->dims[n] <= JAC_FAST_MAX_N && logb <= ((size_t)64 << 20);
    L.w_log[n] = o; if (L.jac_fast[n]) o = align_up(o + logb);
    L.w_lam[n] = o; o = align_up(o + (size_t)c->dims[n] * 4);
    plan_gram(c, n, sm, L.gram_chunks[n], L.gram_cps[n], L.gram_splits[n]);
    size_t pb = sq * L.gram_splits[n];
    if (pb > partial) partial = pb;
    // the tcgen05 kernel (64..256 rows) writes at most this many partial matrices, whatever tensor it is given
    if (c->dims[n] >= GT_MIN_ROWS && c->dims[n] <= GT_MAX_ROWS && sq * kGramTcMaxBlocks > partial) partial = sq * kGramTcMaxBlocks;
  }
  L.w_partial = o; o = align_up(o + partial);
  // refinement sweeps: two buffers for the tensor compressed in all modes but one, and an identity matrix that
  // stands in for the factor of the mode that is left alone when that is one of the two trailing modes
  L.w_hooi0 = L.w_hooi1 = L.w_ident = o; L.hooi_smem = 0;
  if (c->hooi_iters > 0) {
    const uint64_t A = (uint64_t)c->dims[N - 2], B = (uint64_t)c->dims[N - 1], ra = c->ranks[N - 2], rb = c->ranks[N - 1];
    uint64_t per = ra * rb;
    if (A * rb > per) per = A * rb;
    if (ra * B > per) per = ra * B;
    const size_t g1 = tail_blk_geom((int)A, (int)B, (int)A, (int)rb, false).total, g2 = tail_blk_geom((int)A, (int)B, (int)ra, (int)B, false).total;
    L.hooi_smem = (uint32_t)(g1 > g2 ? g1 : g2);
    if (L.hooi_smem > kSmemMax) return TGRAD_ERR_UNSUPPORTED;
    L.w_hooi0 = o; o = align_up(o + (size_t)(S * per) * 8);
    L.w_hooi1 = o; o = align_up(o + (size_t)(S * per) * 8);
    const uint64_t mx = A > B ? A : B;
    L.w_ident = o; o = align_up(o + (size_t)(mx * mx) * 8);
  }
  // low-rank-first composition: G - P_U(G) at full size, from which a refresh selects Omega
  L.w_diag = o; o = align_up(o + 8 * sizeof(double));          // scalars of the diagnostics call
  L.w_rbuf = o;
  if (c->composition == 1) o = align_up(o + (size_t)numel * (c->wg_dtype == TGRAD_C64 ? 8 : 4));
  L.w_total = o;
  return TGRAD_OK;
}

}  // namespace

struct tgrad_state {
  tgrad_config cfg;     // as the kernels see it (a matrix carries a unit mode in the middle)
  int ext_ndim;         // the caller's N
  int mode_map[TGRAD_MAX_NDIM];   // caller's mode -> mode of cfg
  Layout L;
  char* dp;
  char* dw;
  int64_t t;
  bool have_subspace;
  bool basis_valid;     // the persistent block holds factor matrices (of a refresh or an import) a refresh can start from
  bool tabs_stale;      // U^(N-1) changed since the compression kernel's fragment table was built
  int sm_count;
  TailPlan tail;
  // optional per-stage timing
  bool timing;
  int timing_steps;
  cudaEvent_t ev[kTimingRing][kStages + 1];
};

namespace {

#define TG_LAUNCH_CHECK()                                  \
  do {                                                     \
    g_launches.fetch_add(1, std::memory_order_relaxed);    \
    if (cudaPeekAtLastError() != cudaSuccess) return TGRAD_ERR_CUDA; \
  } while (0)

// Launch of a kernel of the step: programmatic dependent launch, so that its blocks are scheduled while the
// previous kernel of the stream drains (every such kernel begins with griddep_chain()).
template <typename... KA, typename... AA>
inline void launch_chained(void (*kern)(KA...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, AA&&... args) {
  cudaLaunchConfig_t lc; memset(&lc, 0, sizeof(lc));
  lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = smem; lc.stream = st;
  cudaLaunchAttribute at; memset(&at, 0, sizeof(at));
  at.id = cudaLaunchAttributeProgrammaticStreamSerialization; at.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &at; lc.numAttrs = 1;
  (void)cudaLaunchKernelEx(&lc, kern, static_cast<KA>(args)...);     // an error stays pending for TG_LAUNCH_CHECK
}

// op: 0 = set attributes, 1 = proj, 2 = back
template <class S>
tgrad_status tail_dispatch(int op, const TailPlan& tp, void* ptr, const TailParams& p, cudaStream_t st) {
  if (op == 0) {
    if (cudaFuncSetAttribute(proj_tail_blk_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(tp.bproj.total > tp.hooi_smem ? tp.bproj.total : tp.hooi_smem)) != cudaSuccess) return TGRAD_ERR_CUDA;
    if (cudaFuncSetAttribute(back_tail_blk_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tp.bback.total) != cudaSuccess) return TGRAD_ERR_CUDA;
    return TGRAD_OK;
  }
  if (op == 2) launch_chained(back_tail_blk_kernel<S>, dim3(tp.grid_bback), dim3(TB_THREADS), tp.bback.total, st, ptr, p, tp.bback);
  else launch_chained(proj_tail_blk_kernel<S>, dim3(tp.grid_bproj), dim3(TB_THREADS), tp.bproj.total, st, ptr, p, tp.bproj);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

tgrad_status tail_any(const tgrad_state* s, int op, void* ptr, const TailParams& p, cudaStream_t st) {
  return s->cfg.wg_dtype == TGRAD_C64    ? tail_dispatch<StoreC64>(op, s->tail, ptr, p, st)
         : s->cfg.wg_dtype == TGRAD_C32H ? tail_dispatch<StoreC32H>(op, s->tail, ptr, p, st)
                                         : tail_dispatch<StoreC32B>(op, s->tail, ptr, p, st);
}

template <int RAT, int KS, int NTW, int TW>
tgrad_status tc_proj_op2(int op, const TailPlan& tp, const void* g, const TailTcParams& P, cudaStream_t st) {
  if (op == 0) {
    return cudaFuncSetAttribute(proj_tail_tc_kernel<RAT, KS, NTW, TW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)tp.gproj.total) == cudaSuccess ? TGRAD_OK : TGRAD_ERR_CUDA;
  }
  launch_chained(proj_tail_tc_kernel<RAT, KS, NTW, TW>, dim3(tp.grid_proj), dim3(32 * PJ_WARPS), tp.gproj.total, st, g, P);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}
template <int RAT, int KS>
tgrad_status tc_proj_op(int op, const TailPlan& tp, const void* g, const TailTcParams& P, cudaStream_t st) {
  // (row tiles per warp, warps per slab): 64 rows -> (2, 4), 32 rows -> (4, 1), 16 rows -> (2, 1)
  if (tp.ntw == 4 && tp.gproj.tps == 1) return tc_proj_op2<RAT, KS, 4, 1>(op, tp, g, P, st);
  if (tp.ntw == 2 && tp.gproj.tps == 4) return tc_proj_op2<RAT, KS, 2, 4>(op, tp, g, P, st);
  if (tp.ntw == 2 && tp.gproj.tps == 1) return tc_proj_op2<RAT, KS, 2, 1>(op, tp, g, P, st);
  return TGRAD_ERR_UNSUPPORTED;
}
template <int RAT, int NS, int NBT>
tgrad_status tc_back_op2(int op, const TailPlan& tp, void* w, const TailTcParams& P, cudaStream_t st) {
  if (op == 0) {
    return cudaFuncSetAttribute(back_tail_tc_kernel<RAT, NS, NBT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)tp.gback.total) == cudaSuccess ? TGRAD_OK : TGRAD_ERR_CUDA;
  }
  launch_chained(back_tail_tc_kernel<RAT, NS, NBT>, dim3(tp.grid_back), dim3(TC_THREADS), tp.gback.total, st, w, P);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}
template <int RAT, int NS>
tgrad_status tc_back_op1(int op, const TailPlan& tp, void* w, const TailTcParams& P, cudaStream_t st) {
  // the common tile counts (trailing extents 16, 17, 32, 33 and those that pad to them) are built in
  switch (tp.gback.nbt) {
    case 4: return tc_back_op2<RAT, NS, 4>(op, tp, w, P, st);
    case 5: return tc_back_op2<RAT, NS, 5>(op, tp, w, P, st);
    case 8: return tc_back_op2<RAT, NS, 8>(op, tp, w, P, st);
    case 9: return tc_back_op2<RAT, NS, 9>(op, tp, w, P, st);
    default: return tc_back_op2<RAT, NS, 0>(op, tp, w, P, st);
  }
}
template <int RAT>
tgrad_status tc_back_op(int op, const TailPlan& tp, void* w, const TailTcParams& P, cudaStream_t st) {
  return tp.back_ns == 2 ? tc_back_op1<RAT, 2>(op, tp, w, P, st) : tc_back_op1<RAT, 1>(op, tp, w, P, st);
}
template <int RAT, int RBT>
tgrad_status th_proj_op(int op, const TailPlan& tp, const void* g, const TailHParams& P, cudaStream_t st) {
  if (op == 0) {
    return cudaFuncSetAttribute(proj_tail_h_kernel<RAT, RBT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)tp.gh.total) == cudaSuccess ? TGRAD_OK : TGRAD_ERR_CUDA;
  }
  launch_chained(proj_tail_h_kernel<RAT, RBT>, dim3(tp.grid_h), dim3(32 * tp.gh.nwarps), tp.gh.total, st, g, P);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}
tgrad_status th_dispatch(int op, const TailPlan& tp, const void* g, const TailHParams& P, cudaStream_t st) {
#define TG_HCASE(RAT_, RBT_) if (tp.h_rat == RAT_ && tp.h_rbt == RBT_) return th_proj_op<RAT_, RBT_>(op, tp, g, P, st);
  TG_HCASE(1, 1) TG_HCASE(2, 1) TG_HCASE(3, 1) TG_HCASE(4, 1) TG_HCASE(1, 2) TG_HCASE(2, 2) TG_HCASE(3, 2) TG_HCASE(4, 2)
#undef TG_HCASE
  return TGRAD_ERR_UNSUPPORTED;
}

template <int RAT, int RBT, int NBT>
tgrad_status th_back_op2(int op, const TailPlan& tp, void* w, const TailHBParams& P, cudaStream_t st) {
  if (op == 0) {
    return cudaFuncSetAttribute(back_tail_h_kernel<RAT, RBT, NBT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)tp.ghb.total) == cudaSuccess ? TGRAD_OK : TGRAD_ERR_CUDA;
  }
  launch_chained(back_tail_h_kernel<RAT, RBT, NBT>, dim3(tp.grid_hb), dim3(32 * tp.ghb.nwarps), tp.ghb.total, st, w, P);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}
template <int RAT, int RBT>
tgrad_status th_back_op(int op, const TailPlan& tp, void* w, const TailHBParams& P, cudaStream_t st) {
  // rows of 65 entries (17 column tiles) have their own instance with the tile loop unrolled
  if (tp.ghb.nbt == 17) return th_back_op2<RAT, RBT, 17>(op, tp, w, P, st);
  return th_back_op2<RAT, RBT, 0>(op, tp, w, P, st);
}
tgrad_status thb_dispatch(int op, const TailPlan& tp, void* w, const TailHBParams& P, cudaStream_t st) {
#define TG_HCASE(RAT_, RBT_) if (tp.h_rat == RAT_ && tp.h_rbt == RBT_) return th_back_op<RAT_, RBT_>(op, tp, w, P, st);
  TG_HCASE(1, 1) TG_HCASE(2, 1) TG_HCASE(3, 1) TG_HCASE(4, 1) TG_HCASE(1, 2) TG_HCASE(2, 2) TG_HCASE(3, 2) TG_HCASE(4, 2)
#undef TG_HCASE
  return TGRAD_ERR_UNSUPPORTED;
}

// op: 0 = set attributes (both kernels), 1 = proj, 2 = back
tgrad_status tc_dispatch(int op, const TailPlan& tp, void* ptr, const TailTcParams& P, cudaStream_t st) {
#define TG_TCASE(RAT_)                                                                           \
  if (tp.rat == RAT_) {                                                                          \
    if (op == 0 || op == 2) {                                                                    \
      tgrad_status r = tc_back_op<RAT_>(op, tp, ptr, P, st);                                     \
      if (op == 2 || r != TGRAD_OK) return r;                                                    \
    }                                                                                            \
    if (tp.ks == 4) return tc_proj_op<RAT_, 4>(op, tp, ptr, P, st);                              \
    if (tp.ks == 5) return tc_proj_op<RAT_, 5>(op, tp, ptr, P, st);                              \
    if (tp.ks == 8) return tc_proj_op<RAT_, 8>(op, tp, ptr, P, st);                              \
    if (tp.ks == 9) return tc_proj_op<RAT_, 9>(op, tp, ptr, P, st);                              \
    return TGRAD_ERR_UNSUPPORTED;                                                                \
  }
  TG_TCASE(1) TG_TCASE(2)
#undef TG_TCASE
  return TGRAD_ERR_UNSUPPORTED;
}

tgrad_status plan_tail(tgrad_state* s) {
  const tgrad_config& c = s->cfg;
  const int N = c.ndim;
  const int A = (int)c.dims[N - 2], B = (int)c.dims[N - 1], ra = c.ranks[N - 2], rb = c.ranks[N - 1];
  TailPlan& tp = s->tail;
  const size_t kMax = 227 * 1024;
  tp.bproj = tail_blk_geom(A, B, ra, rb, false);
  tp.bback = tail_blk_geom(A, B, ra, rb, true);
  tp.hooi_smem = s->L.hooi_smem;
  if (tp.bproj.total > kMax || tp.bback.total > kMax) return TGRAD_ERR_UNSUPPORTED;   // a trailing A x B slab does not fit in shared memory
  uint64_t S = s->L.numel / ((uint64_t)A * B);
  {
    const int pp = (int)(kMax / (tp.bproj.total + 1024)), pb = (int)(kMax / (tp.bback.total + 1024));
    const uint64_t gp = (uint64_t)s->sm_count * (pp < 1 ? 1 : (pp > 8 ? 8 : pp));
    const uint64_t gb = (uint64_t)s->sm_count * (pb < 1 ? 1 : (pb > 8 ? 8 : pb));
    tp.grid_bproj = (int)(S < gp ? S : gp);
    tp.grid_bback = (int)(S < gb ? S : gb);
  }
  TailParams dummy; memset(&dummy, 0, sizeof(dummy));
  tgrad_status r = tail_any(s, 0, nullptr, dummy, 0);
  if (r != TGRAD_OK) return r;
  // fast path
  tp.tc = false;
  const int rat = (ra + 7) / 8, ksn = tc_ksteps(B);
  const int ks = ksn <= 4 ? 4 : ksn == 5 ? 5 : ksn <= 8 ? 8 : ksn == 9 ? 9 : 0;
  const double dec = 1.0 - (double)c.lr * (double)c.weight_decay;
  if (c.wg_dtype == TGRAD_C64 && (A == 16 || A == 32 || A == 64) && rat <= 2 && rb <= 8 && ks && dec > 0.0) {
    tp.rat = rat; tp.ks = ks;
    // compression kernel: blocks of 4 warps; two row tiles per warp for 64-row and 16-row slabs, four for 32-row
    // slabs (measured: two tiles per warp there, two warps per slab, 218 against 200 us on 64x64x32x32x17)
    tp.pjw = 4; tp.ntw = (A == 64) ? 2 : (A == 32 ? 4 : 2);
    tp.back_ns = ((uint64_t)A * B * 8 <= 8192) ? 2 : 1;      // small slabs: two per warp and iteration
    const int pj_blocks = 4;     // resident blocks per SM
    const uint32_t pj_smem = (227u * 1024u) / pj_blocks - 1024u;
    if (proj_tc_geom(A, B, rat, (uint32_t)S, tp.ntw, tp.pjw, pj_smem, tp.gproj) && tail_tc_geom(true, A, B, rat, (uint32_t)S, tp.back_ns, tp.gback)) {
      const uint32_t cap = 2u * (uint32_t)s->sm_count, pcap = (uint32_t)pj_blocks * (uint32_t)s->sm_count;
      tp.grid_proj = (int)(tp.gproj.ngroups < pcap ? tp.gproj.ngroups : pcap);
      tp.grid_back = (int)(tp.gback.ngroups < cap ? tp.gback.ngroups : cap);
      TailTcParams dm; memset(&dm, 0, sizeof(dm));
      if (tc_dispatch(0, tp, nullptr, dm, 0) == TGRAD_OK) tp.tc = true;
    }
  }
  // half storage: compression with fp16 MMAs on the stored values
  tp.th = false;
  if (c.wg_dtype == TGRAD_C32H && tail_h_geom(A, B, ra, rb, tp.gh)) {
    tp.h_rat = (ra + 7) / 8; tp.h_rbt = (rb + 7) / 8;
    tp.grid_h = (int)(S < (uint64_t)s->sm_count ? S : (uint64_t)s->sm_count);
    TailHParams dm; memset(&dm, 0, sizeof(dm));
    if (th_dispatch(0, tp, nullptr, dm, 0) == TGRAD_OK) tp.th = true;
  }
  tp.thb = false;
  if (c.wg_dtype == TGRAD_C32H && tail_hb_geom(A, B, ra, rb, tp.ghb)) {
    tp.h_rat = (ra + 7) / 8; tp.h_rbt = (rb + 7) / 8;
    tp.grid_hb = (int)(S < (uint64_t)s->sm_count ? S : (uint64_t)s->sm_count);
    TailHBParams dm; memset(&dm, 0, sizeof(dm));
    if (thb_dispatch(0, tp, nullptr, dm, 0) == TGRAD_OK) tp.thb = true;
  }
  return TGRAD_OK;
}

AdamScalars adam_scalars(const tgrad_config& c, int64_t t) {
  AdamScalars a;
  a.beta1 = c.beta1; a.beta2 = c.beta2;
  a.omb1 = 1.0f - c.beta1; a.omb2 = 1.0f - c.beta2;
  float c1 = (float)(1.0 - std::pow((double)c.beta1, (double)(t + 1)));
  float c2 = (float)(1.0 - std::pow((double)c.beta2, (double)(t + 1)));
  a.inv_c1 = 1.0f / c1; a.inv_c2 = 1.0f / c2;
  a.eps = c.eps;
  return a;
}

tgrad_status build_slab_ptr(tgrad_state* s, cudaStream_t st) {
  const Layout& L = s->L;
  slab_ptr_kernel<<<(L.nslab + 1 + 255) / 256, 256, 0, st>>>(reinterpret_cast<const uint32_t*>(s->dp + L.p_omega),
                                                              (uint32_t)s->cfg.k, L.E, L.nslab,
                                                              reinterpret_cast<uint32_t*>(s->dp + L.p_slab));
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

#define TG_TRY(x) do { tgrad_status _s = (x); if (_s != TGRAD_OK) return _s; } while (0)

tgrad_status mode_product(bool conj_t, const cf* in, cf* out, const cf* U, uint64_t O, int M, int K, uint64_t C,
                          int r_n, int sm_count, cudaStream_t st);

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link against the driver.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

template <class S> struct GramTcFmt;
template <> struct GramTcFmt<StoreC64> { static constexpr int fmt = 2; static constexpr CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT32; };
template <> struct GramTcFmt<StoreC32H> { static constexpr int fmt = 0; static constexpr CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT16; };
template <> struct GramTcFmt<StoreC32B> { static constexpr int fmt = 1; static constexpr CUtensorMapDataType dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16; };

// The same on the tcgen05 kernel: a rank-3 tensor map (2C reals, In rows, O blocks) over this GPU's own memory.
template <class S>
tgrad_status launch_gram_tc(tgrad_state* s, const void* x, int In, uint64_t O, uint64_t C, const GramTcPlan& pl, cf* A,
                            cudaStream_t st) {
  EncodeTiledFn enc = encode_tiled_fn();
  if (!enc) return TGRAD_ERR_CUDA;
  constexpr int fmt = GramTcFmt<S>::fmt;
  const uint64_t real_bytes = S::kBytes / 2;
  GramTcParams gp;
  gp.ld = In; gp.partial = reinterpret_cast<cf*>(s->dw + s->L.w_partial);
  gp.flags = reinterpret_cast<int*>(s->dp + s->L.p_flags);
  for (int i = 0; i < pl.nlaunch; ++i) {
    const GramTcLaunch& l = pl.l[i];
    CUtensorMap tm;
    const cuuint64_t dims[3] = {2 * C, (cuuint64_t)In, O};
    const cuuint64_t strides[2] = {C * S::kBytes, (cuuint64_t)In * C * S::kBytes};
    const cuuint32_t box[3] = {(cuuint32_t)(GT_ROW_BYTES / real_bytes), (cuuint32_t)l.rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (enc(&tm, GramTcFmt<S>::dt, 3, const_cast<void*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return TGRAD_ERR_CUDA;
    gp.In = l.In; gp.rows = l.rows; gp.row0 = l.row0; gp.a_min = l.a_min; gp.stages = l.stages; gp.kt = l.kt;
    gp.tiles_per_o = l.tiles_per_o; gp.tiles_total = l.tiles_total; gp.tiles_per_split = l.per;
    gp.group_tiles = (uint32_t)(32 / l.kt);
    size_t smem = gram_tc_smem(l.rows, l.stages, l.kt);
    if (smem < ((size_t)120 << 10)) smem = (size_t)120 << 10;   // one block per SM: each takes all of the tensor memory
    gram_tc_kernel<fmt><<<l.splits, GT_THREADS, smem, st>>>(tm, gp); TG_LAUNCH_CHECK();
  }
  gram_reduce_kernel<<<(In * In + GRR_E - 1) / GRR_E, GRR_E * GRR_G, 0, st>>>(gp.partial, pl.splits, In, A); TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

// A = X_(n) X_(n)^H for a tensor seen as [O][In][C] (storage S), split-K partial sums reduced in a fixed order.
template <class S>
tgrad_status launch_gram(tgrad_state* s, const void* x, int In, uint64_t O, uint64_t C, uint32_t chunks, uint32_t cps,
                         int splits, cf* A, cudaStream_t st) {
  const GramTcPlan pl = plan_gram_tc(In, O, C, S::kBytes, s->sm_count);
  if (pl.ok && (reinterpret_cast<uintptr_t>(x) & 15) == 0) return launch_gram_tc<S>(s, x, In, O, C, pl, A, st);
  cf* partial = reinterpret_cast<cf*>(s->dw + s->L.w_partial);
  const int T = (In + GR_T - 1) / GR_T;
  dim3 grid(T * T, splits);
  // long contractions average the TF32 input rounding away; short ones get the split-precision products
  const bool full = (In % GR_T) == 0;
#define TG_GRAM(SPLIT_, FULL_)                                                                                   \
  gram_partial_kernel<S, SPLIT_, FULL_><<<grid, GR_THREADS, GR_SMEM, st>>>(x, In, (uint32_t)O, (uint32_t)C, chunks, \
                                                                          cps, partial)
  if (O * C >= 16384) { if (full) TG_GRAM(false, true); else TG_GRAM(false, false); }
  else { if (full) TG_GRAM(true, true); else TG_GRAM(true, false); }
#undef TG_GRAM
  TG_LAUNCH_CHECK();
  gram_reduce_kernel<<<(In * In + GRR_E - 1) / GRR_E, GRR_E * GRR_G, 0, st>>>(partial, splits, In, A); TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

// U^(m) <- eigenvectors of the r_m largest eigenvalues of the Gram matrix stored for mode m, for the listed modes:
// subspace iteration where the rank leaves room for guard columns (started from the stored factor if `warm`), then
// the full Jacobi diagonalisation, which returns at once for the modes the iteration has delivered.
tgrad_status solve_modes(tgrad_state* s, const int* modes, int nm, bool warm, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  int* flags = reinterpret_cast<int*>(s->dp + L.p_flags);
  JacobiParams jp; memset(&jp, 0, sizeof(jp));
  JacobiFastParams fp; memset(&fp, 0, sizeof(fp));
  SubspaceParams sp; memset(&sp, 0, sizeof(sp));
  size_t sub_bytes = 0;
  int nslow = 0;
  for (int i = 0; i < nm; ++i) {
    const int m = modes[i];
    // this mode's factor is not written yet (the eigensolvers below read the word); only this call's modes are
    // touched: another group of modes may be in flight on another stream
    if (cudaMemsetAsync(flags + SUB_DONE + m, 0, sizeof(int), st) != cudaSuccess) return TGRAD_ERR_CUDA;
    const int In = (int)c.dims[m];
    cf* A = reinterpret_cast<cf*>(s->dw + L.w_gram[m]);
    {
      int R = 0; bool zsm = false;
      if (sub_eligible(In, c.ranks[m], R, zsm)) {
        SubspaceMode& sm_ = sp.mode[sp.nmodes++];
        sm_.A = A; sm_.U = reinterpret_cast<cf*>(s->dp + L.p_factor[m]);
        sm_.Zg = reinterpret_cast<cf*>(s->dw + L.w_v[m]);
        sm_.n = In; sm_.r = c.ranks[m]; sm_.R = R; sm_.index = m; sm_.z_in_smem = zsm ? 1 : 0;
        const size_t b = sub_smem(In, R, zsm);
        if (b > sub_bytes) sub_bytes = b;
      }
    }
    if (L.jac_fast[m]) {
      JacobiFastMode& fm = fp.mode[fp.nmodes++];
      fm.A = A;
      fm.work = reinterpret_cast<cf*>(s->dw + L.w_jac[m]);
      fm.log = reinterpret_cast<float4*>(s->dw + L.w_log[m]);
      fm.lam = reinterpret_cast<float*>(s->dw + L.w_lam[m]);
      fm.V = reinterpret_cast<cf*>(s->dw + L.w_v[m]);
      fm.U = reinterpret_cast<cf*>(s->dp + L.p_factor[m]);
      fm.n = In; fm.r = c.ranks[m]; fm.index = m; fm.row0 = fp.total_rows;
      fp.total_rows += In;
      if (In > fp.row_stride) fp.row_stride = In;
    } else {
      JacobiMode& jm = jp.mode[nslow];
      jp.index[nslow++] = m;
      jm.A = reinterpret_cast<cf*>(s->dw + L.w_jac[m]);
      jm.V = reinterpret_cast<cf*>(s->dw + L.w_v[m]);
      jm.U = reinterpret_cast<cf*>(s->dp + L.p_factor[m]);
      jm.n = In; jm.r = c.ranks[m];
      if (cudaMemcpyAsync(s->dw + L.w_jac[m], A, (size_t)In * In * 8, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return TGRAD_ERR_CUDA;
    }
  }
  const int max_sweeps = c.jacobi_max_sweeps > 0 ? c.jacobi_max_sweeps : 30;
  const float tol = c.jacobi_tol > 0.f ? c.jacobi_tol : 1e-6f;
  if (sp.nmodes) {
    sp.warm = warm ? 1 : 0;
    sp.max_sweeps = max_sweeps; sp.tol = tol; sp.flags = flags;
    subspace_kernel<<<sp.nmodes, SUB_THREADS, sub_bytes, st>>>(sp); TG_LAUNCH_CHECK();
  }
  if (nslow) {
    jp.max_sweeps = max_sweeps; jp.tol = tol; jp.flags = flags;
    jacobi_kernel<<<nslow, JAC_THREADS, 0, st>>>(jp); TG_LAUNCH_CHECK();
  }
  if (fp.nmodes) {
    fp.max_sweeps = max_sweeps; fp.tol = tol; fp.flags = flags;
    // the sweeps: modes whose matrix fits in shared memory in one launch, the larger ones (matrix in L2) in another
    JacobiFastParams fs = fp, fg = fp;
    fs.nmodes = fg.nmodes = 0;
    size_t smem_s = 0, smem_g = 0;
    for (int i = 0; i < fp.nmodes; ++i) {
      const int n = fp.mode[i].n;
      if (n <= JAC_SMEM_MAX_N) { fs.mode[fs.nmodes++] = fp.mode[i]; const size_t b = jac_sweeps_smem(n, true); if (b > smem_s) smem_s = b; }
      else { fg.mode[fg.nmodes++] = fp.mode[i]; const size_t b = jac_sweeps_smem(n, false); if (b > smem_g) smem_g = b; }
    }
    if (fg.nmodes) { jacobi_sweeps_kernel<false><<<fg.nmodes, JAC_THREADS, smem_g, st>>>(fg); TG_LAUNCH_CHECK(); }
    if (fs.nmodes) { jacobi_sweeps_kernel<true><<<fs.nmodes, JAC_THREADS, smem_s, st>>>(fs); TG_LAUNCH_CHECK(); }
    fp.row_stride = (fp.row_stride + 1) & ~1;
    const size_t vsm = (size_t)8 * fp.row_stride * sizeof(cf);
    if (fp.row_stride <= 192) jacobi_vectors_kernel<3, 4><<<(fp.total_rows + 7) / 8, 256, vsm, st>>>(fp);
    else jacobi_vectors_kernel<4, 2><<<(fp.total_rows + 7) / 8, 256, vsm, st>>>(fp);
    TG_LAUNCH_CHECK();
    jacobi_factors_kernel<<<fp.nmodes, JAC_THREADS, 0, st>>>(fp); TG_LAUNCH_CHECK();
  }
  return TGRAD_OK;
}

// Omega <- the k entries of x with the largest selection keys (ascending), their values into the gather buffer.
template <class S>
tgrad_status select_omega(tgrad_state* s, const void* x, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const uint32_t n = (uint32_t)L.numel, k = (uint32_t)c.k;
  int* flags = reinterpret_cast<int*>(s->dp + L.p_flags);
  uint32_t* omega = reinterpret_cast<uint32_t*>(s->dp + L.p_omega);
  cf* g_s = reinterpret_cast<cf*>(s->dw + L.w_gs);
  SelState* sel = reinterpret_cast<SelState*>(s->dw + L.w_sel);
  uint32_t* hist = reinterpret_cast<uint32_t*>(s->dw + L.w_hist);
  uint32_t* blk_gt = reinterpret_cast<uint32_t*>(s->dw + L.w_blk);
  uint32_t* blk_eq = blk_gt + L.nblk;
  SelKey kp;
  kp.seed_lo = (uint32_t)(c.seed & 0xffffffffull); kp.seed_hi = (uint32_t)(c.seed >> 32);
  kp.epoch = (uint32_t)(s->t / c.T); kp.strategy = c.sparse_strategy;
  // candidate keys of the threshold bucket: in the two buffers of the compressed tensor, which nothing uses while
  // Omega is being selected; runs of candidates per block of kChunk entries behind the per-block counts
  uint32_t* cand = reinterpret_cast<uint32_t*>(s->dw + L.w_bufa);
  uint64_t cap64 = (uint64_t)(L.w_bufb + L.tsize * 8 - L.w_bufa) / 4;
  if (cap64 > n / 4) cap64 = n / 4;
  uint32_t* cand_start = blk_eq + L.nblk;
  uint32_t* cand_cnt = cand_start + L.nblk;
  if (cudaMemsetAsync(hist, 0, 3 * kSelMaxBins * 4, st) != cudaSuccess) return TGRAD_ERR_CUDA;
  sel_init_kernel<<<1, 1, 0, st>>>(sel, k, (uint32_t)cap64); TG_LAUNCH_CHECK();
  uint64_t want = ((uint64_t)n + 511) / 512;
  int hgrid = (int)(want < (uint64_t)s->sm_count * 8 ? want : (uint64_t)s->sm_count * 8);
  const bool topk = c.sparse_strategy == 0;
  for (int pass = 0; pass < 3; ++pass) {
    // passes 1 and 2: one of the two histogram kernels returns at once (decided on the device by the first pick)
    if (topk) sel_hist_kernel<S, true><<<hgrid, 512, 0, st>>>(x, n, pass, sel, hist + pass * kSelMaxBins, flags, kp);
    else sel_hist_kernel<S, false><<<hgrid, 512, 0, st>>>(x, n, pass, sel, hist + pass * kSelMaxBins, flags, kp);
    TG_LAUNCH_CHECK();
    if (pass > 0) { sel_hist_keys_kernel<<<2 * s->sm_count, 512, 0, st>>>(cand, pass, sel, hist + pass * kSelMaxBins); TG_LAUNCH_CHECK(); }
    sel_pick_kernel<<<1, 1024, 0, st>>>(hist + pass * kSelMaxBins, pass, sel); TG_LAUNCH_CHECK();
    if (pass == 0) {
      if (topk) sel_gather_kernel<S, true><<<L.nblk, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, cand, cand_start, cand_cnt, kp);
      else sel_gather_kernel<S, false><<<L.nblk, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, cand, cand_start, cand_cnt, kp);
      TG_LAUNCH_CHECK();
    }
  }
  const uint32_t cgrid = L.nblk < (uint32_t)s->sm_count * 8 ? L.nblk : (uint32_t)s->sm_count * 8;
  if (topk) sel_count_kernel<S, true><<<cgrid, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, kp);
  else sel_count_kernel<S, false><<<cgrid, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, kp);
  TG_LAUNCH_CHECK();
  sel_count_cand_kernel<<<(L.nblk + 255) / 256, 256, 0, st>>>(cand, cand_start, cand_cnt, sel, blk_gt, blk_eq, L.nblk); TG_LAUNCH_CHECK();
  sel_scan_kernel<<<1, 1024, 0, st>>>(blk_gt, blk_eq, L.nblk); TG_LAUNCH_CHECK();
  if (topk) sel_compact_kernel<S, true><<<L.nblk, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, omega, g_s, k, kp);
  else sel_compact_kernel<S, false><<<L.nblk, kChunkThreads, 0, st>>>(x, n, sel, blk_gt, blk_eq, omega, g_s, k, kp);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

// ---- pieces of a step, shared with the refresh of the low-rank-first composition ----

// Geometry, factor and index pointers and the update scalars of the two streaming kernels.
TailParams tail_params(const tgrad_state* s) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  const int A = (int)c.dims[N - 2], B = (int)c.dims[N - 1], ra = c.ranks[N - 2], rb = c.ranks[N - 1];
  TailParams p; memset(&p, 0, sizeof(p));
  p.A = A; p.B = B; p.Bs = B | 1; p.ra = ra; p.rb = rb; p.ras = ra | 1;
  p.E = (uint32_t)((uint64_t)A * B); p.nslab = (uint32_t)(L.numel / p.E);
  p.Ua = reinterpret_cast<const cf*>(s->dp + L.p_factor[N - 2]);
  p.Ub = reinterpret_cast<const cf*>(s->dp + L.p_factor[N - 1]);
  p.omega = reinterpret_cast<const uint32_t*>(s->dp + L.p_omega);
  p.slab_ptr = reinterpret_cast<const uint32_t*>(s->dp + L.p_slab);
  p.k = (int)c.k;
  p.m_s = reinterpret_cast<cf*>(s->dp + L.p_ms);
  p.v_s = reinterpret_cast<float*>(s->dp + L.p_vs);
  p.n_s = reinterpret_cast<cf*>(s->dw + L.w_ns);
  p.g_s = reinterpret_cast<cf*>(s->dw + L.w_gs);
  p.s_low = (float)((double)c.lr * (double)c.alpha);
  p.s_sparse = (float)((double)c.lr * (double)c.lambda);
  p.decay = (float)(1.0 - (double)c.lr * (double)c.weight_decay);
  return p;
}

// Compression of the two trailing modes of the tensor at d_grad into p.t, with the sparse gather if p.k > 0.
tgrad_status run_proj_tail(tgrad_state* s, const void* d_grad, const TailParams& p, cudaStream_t st) {
  const Layout& L = s->L;
  int* flags = reinterpret_cast<int*>(s->dp + L.p_flags);
  if (s->tail.tc) {
    TailTcParams mp; mp.flags = flags; mp.s_sparse_pre = 0.f;
    mp.p = p; mp.g = s->tail.gproj;
    float4* tab = reinterpret_cast<float4*>(s->dp + L.p_u2tab);
    if (s->tabs_stale) {
      const int n_ent = (p.A / 8) * s->tail.rat * 32;
      proj_u2tab_kernel<<<(n_ent + 127) / 128, 128, 0, st>>>(p.Ua, p.A, p.ra, s->tail.rat, tab);
      TG_LAUNCH_CHECK();
      s->tabs_stale = false;
    }
    mp.u2tab = tab;
    return tc_dispatch(1, s->tail, const_cast<void*>(d_grad), mp, st);
  }
  if (s->tail.th) {
    TailHParams hp; hp.p = p; hp.g = s->tail.gh; hp.flags = flags;
    return th_dispatch(1, s->tail, d_grad, hp, st);
  }
  return tail_any(s, 1, const_cast<void*>(d_grad), p, st);
}

// Reconstruction of the two trailing modes from p.t, fused with the update of the tensor at d_weight:
// W <- decay W - s_low D, then W[Omega] -= s_sparse N_S if p.k > 0.
tgrad_status run_back_tail(tgrad_state* s, void* d_weight, const TailParams& p, cudaStream_t st) {
  int* flags = reinterpret_cast<int*>(s->dp + s->L.p_flags);
  if (s->tail.tc) {
    TailTcParams mp; mp.flags = flags; mp.u2tab = nullptr;
    const tgrad_config& c = s->cfg;
    mp.s_sparse_pre = (float)((double)c.lr * (double)c.lambda / (1.0 - (double)c.lr * (double)c.weight_decay));
    mp.p = p; mp.g = s->tail.gback;
    return tc_dispatch(2, s->tail, d_weight, mp, st);
  }
  if (s->tail.thb) {
    TailHBParams hp; hp.p = p; hp.g = s->tail.ghb; hp.flags = flags;
    return thb_dispatch(2, s->tail, d_weight, hp, st);
  }
  return tail_any(s, 2, d_weight, p, st);
}

// Whether the first mode's two products and the AdamUpdate of the core run as one launch.
bool chain_fused(const tgrad_config& c) {
  const int N = c.ndim;
  uint64_t c_first = (uint64_t)c.ranks[N - 2] * c.ranks[N - 1];
  for (int q = 1; q <= N - 3; ++q) c_first *= c.ranks[q];
  return c.dims[0] <= SW_MAX_I && c.ranks[0] <= SW_MAX_R &&
         c_first * (uint64_t)c.dims[0] * (uint64_t)c.ranks[0] <= ((uint64_t)64 << 20);
}

// Compression of modes N-2 .. last (last = 1: the first mode is left for the fused launch; last = 0: down to the
// core, which lands in the core buffer), starting from the tail-contracted tensor in the first chain buffer.
// *out = where the result is, *Cout = its trailing extent.
tgrad_status compress_chain(tgrad_state* s, int last, cf** out, uint64_t* Cout, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  cf* cur = reinterpret_cast<cf*>(s->dw + L.w_bufa);
  cf* nxt = reinterpret_cast<cf*>(s->dw + L.w_bufb);
  cf* core = reinterpret_cast<cf*>(s->dw + L.w_core);
  uint64_t C = (uint64_t)c.ranks[N - 2] * c.ranks[N - 1];
  for (int m = N - 3; m >= last; --m) {
    uint64_t O = 1;
    for (int q = 0; q < m; ++q) O *= c.dims[q];
    cf* dst = (m == 0) ? core : nxt;
    TG_TRY(mode_product(true, cur, dst, reinterpret_cast<const cf*>(s->dp + L.p_factor[m]), O, c.ranks[m],
                        (int)c.dims[m], C, c.ranks[m], s->sm_count, st));
    C *= c.ranks[m];
    if (m == 0) { cur = core; break; }
    cf* tmp = cur; cur = nxt; nxt = tmp;
  }
  *out = cur; *Cout = C;
  return TGRAD_OK;
}

// Reconstruction of modes mfirst .. N-3 (mfirst = 0 from a core-shaped tensor, 1 after the fused launch) into the
// chain buffers, alternating from buffer `which`; *out = the tensor [I_1 .. I_{N-2}][r_{N-1}][r_N].
tgrad_status expand_chain(tgrad_state* s, const cf* src, int mfirst, int which, const cf** out, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  cf* bufs[2] = {reinterpret_cast<cf*>(s->dw + L.w_bufa), reinterpret_cast<cf*>(s->dw + L.w_bufb)};
  uint64_t O = 1;
  for (int q = 0; q < mfirst; ++q) O *= c.dims[q];
  for (int m = mfirst; m <= N - 3; ++m) {
    uint64_t Cm = (uint64_t)c.ranks[N - 2] * c.ranks[N - 1];
    for (int q = m + 1; q <= N - 3; ++q) Cm *= c.ranks[q];
    cf* dst = bufs[which];
    TG_TRY(mode_product(false, src, dst, reinterpret_cast<const cf*>(s->dp + L.p_factor[m]), O, (int)c.dims[m],
                        c.ranks[m], Cm, c.ranks[m], s->sm_count, st));
    O *= c.dims[m];
    src = dst; which ^= 1;
  }
  *out = src;
  return TGRAD_OK;
}

// g_s[j] -= P_U(G)[Omega[j]], with P_U(G) given down to the two trailing modes: t[slab][ja][jb].
__global__ void lowrank_at_omega_kernel(cf* __restrict__ g_s, const uint32_t* __restrict__ omega, uint32_t k,
                                        const cf* __restrict__ t, const cf* __restrict__ Ua, const cf* __restrict__ Ub,
                                        int A, int B, int ra, int rb, uint32_t E) {
  const uint32_t j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= k) return;
  const uint32_t w = omega[j], slab = w / E, loc = w - slab * E;
  const int a = (int)(loc / (uint32_t)B), b = (int)(loc - (uint32_t)a * (uint32_t)B);
  const cf* ts = t + (size_t)slab * ra * rb;
  cf acc = make_float2(0.f, 0.f);
  for (int ja = 0; ja < ra; ++ja) {
    cf row = make_float2(0.f, 0.f);
    for (int jb = 0; jb < rb; ++jb) cfma(row, ts[ja * rb + jb], Ub[b * rb + jb]);
    cfma(acc, row, Ua[a * ra + ja]);
  }
  cf v = g_s[j];
  v.x -= acc.x; v.y -= acc.y;
  g_s[j] = v;
}

// ---- diagnostics (not on the timed path) ----
// *acc += sum |x_i|^2 over n complex entries of storage S, in double
template <class S>
__global__ void diag_sumsq_kernel(const void* __restrict__ x, uint64_t n, double* __restrict__ acc) {
  __shared__ double sh[8];
  double sum = 0.0;
  for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
    const cf v = S::load(x, i);
    sum += (double)v.x * v.x + (double)v.y * v.y;
  }
  for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    atomicAdd(acc, t);
  }
}
// *defect = max(*defect, max_{a,b} |(U^H U - I)[a][b]|) for an n x r factor (the maximum of non-negative floats is
// the maximum of their bit patterns)
__global__ void diag_ortho_kernel(const cf* __restrict__ U, int n, int r, unsigned int* __restrict__ defect) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= r * r) return;
  const int a = idx / r, b = idx - a * r;
  cf acc = make_float2(0.f, 0.f);
  for (int i = 0; i < n; ++i) cfma_conj(acc, U[(size_t)i * r + b], U[(size_t)i * r + a]);
  if (a == b) acc.x -= 1.f;
  atomicMax(defect, __float_as_uint(fmaxf(fabsf(acc.x), fabsf(acc.y))));
}

__global__ void identity_kernel(cf* __restrict__ m, int n) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < n * n) m[idx] = make_float2((idx / n) == (idx % n) ? 1.f : 0.f, 0.f);
}

// One mode update of the refinement: Y = R x_{q != m} U^(q)H through the general streaming kernel (the two trailing
// modes, the identity standing in for U^(m) if m is one of them) and the chain of mode products (mode m left out),
// then A = Y_(m) Y_(m)^H and its leading eigenvectors, started from the current U^(m).  `d_grad` holds the residual
// (the entries at Omega are zero during a refresh).
template <class S>
tgrad_status hooi_mode_update(tgrad_state* s, int m, const void* d_grad, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  const int A = (int)c.dims[N - 2], B = (int)c.dims[N - 1];
  cf* ident = reinterpret_cast<cf*>(s->dw + L.w_ident);
  int ra = c.ranks[N - 2], rb = c.ranks[N - 1];
  const cf* Ua = reinterpret_cast<const cf*>(s->dp + L.p_factor[N - 2]);
  const cf* Ub = reinterpret_cast<const cf*>(s->dp + L.p_factor[N - 1]);
  if (m == N - 2) { identity_kernel<<<(A * A + 255) / 256, 256, 0, st>>>(ident, A); TG_LAUNCH_CHECK(); Ua = ident; ra = A; }
  if (m == N - 1) { identity_kernel<<<(B * B + 255) / 256, 256, 0, st>>>(ident, B); TG_LAUNCH_CHECK(); Ub = ident; rb = B; }
  TailParams p; memset(&p, 0, sizeof(p));
  p.A = A; p.B = B; p.Bs = B | 1; p.ra = ra; p.rb = rb; p.ras = ra | 1;
  p.E = (uint32_t)((uint64_t)A * B); p.nslab = (uint32_t)(L.numel / p.E);
  p.Ua = Ua; p.Ub = Ub; p.k = 0;
  cf* cur = reinterpret_cast<cf*>(s->dw + L.w_hooi0);
  cf* nxt = reinterpret_cast<cf*>(s->dw + L.w_hooi1);
  p.t = cur;
  const TailBlkGeom G = tail_blk_geom(A, B, ra, rb, false);
  {
    const int per_sm = (int)(kSmemMax / (G.total + 1024));
    const uint64_t cap = (uint64_t)s->sm_count * (per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm));
    const unsigned grid = (unsigned)(p.nslab < cap ? p.nslab : cap);
    proj_tail_blk_kernel<S><<<grid, TB_THREADS, G.total, st>>>(d_grad, p, G); TG_LAUNCH_CHECK();
  }
  // leading modes N-3 .. 0, mode m left as it is; the tensor is [d_0 .. d_{N-3}][ra][rb] with d_q shrinking to r_q
  uint64_t C = (uint64_t)ra * rb;
  for (int q = N - 3; q >= 0; --q) {
    if (q == m) { C *= (uint64_t)c.dims[q]; continue; }
    uint64_t O = 1;
    for (int z = 0; z < q; ++z) O *= c.dims[z];
    TG_TRY(mode_product(true, cur, nxt, reinterpret_cast<const cf*>(s->dp + L.p_factor[q]), O, c.ranks[q], (int)c.dims[q],
                        C, c.ranks[q], s->sm_count, st));
    C *= (uint64_t)c.ranks[q];
    cf* tmp = cur; cur = nxt; nxt = tmp;
  }
  // Gram matrix over mode m of Y, whose extents are r_q for q != m
  uint64_t Oy = 1, Cy = 1;
  for (int q = 0; q < m; ++q) Oy *= (uint64_t)c.ranks[q];
  for (int q = m + 1; q < N; ++q) Cy *= (uint64_t)c.ranks[q];
  uint32_t chunks, cps; int splits;
  plan_gram_dims((int)c.dims[m], Oy, Cy, 148, chunks, cps, splits);
  if (splits > L.gram_splits[m]) {          // the scratch of the partial sums was sized for the full tensor's plan
    const uint64_t per = (chunks + (uint64_t)L.gram_splits[m] - 1) / (uint64_t)L.gram_splits[m];
    cps = (uint32_t)per; splits = (int)((chunks + per - 1) / per);
  }
  TG_TRY(launch_gram<StoreC64>(s, cur, (int)c.dims[m], Oy, Cy, chunks, cps, splits, reinterpret_cast<cf*>(s->dw + L.w_gram[m]), st));
  return solve_modes(s, &m, 1, true, st);
}

// One side stream per device on which the eigenvectors of the leading modes are computed while the Gram matrices of
// the trailing modes are still being accumulated on the caller's stream (the eigensolvers keep one SM per mode busy,
// the Gram kernels all of them).  Created at the first refresh on the device and kept for the life of the process.
struct RefreshStreams {
  std::mutex mu;
  bool ready = false, failed = false;
  cudaStream_t side;
  cudaEvent_t fork, join;
};
RefreshStreams g_refresh[64];
RefreshStreams* refresh_streams() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  RefreshStreams* r = &g_refresh[dev];
  std::lock_guard<std::mutex> lock(r->mu);
  if (!r->ready && !r->failed) {
    const bool ok = cudaStreamCreateWithFlags(&r->side, cudaStreamNonBlocking) == cudaSuccess &&
                    cudaEventCreateWithFlags(&r->fork, cudaEventDisableTiming) == cudaSuccess &&
                    cudaEventCreateWithFlags(&r->join, cudaEventDisableTiming) == cudaSuccess;
    r->ready = ok; r->failed = !ok;
  }
  return r->ready ? r : nullptr;      // nullptr: everything on the caller's stream
}

template <class S>
tgrad_status refresh_impl(tgrad_state* s, void* d_grad, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  const uint32_t n = (uint32_t)L.numel, k = (uint32_t)c.k;
  int* flags = reinterpret_cast<int*>(s->dp + L.p_flags);
  uint32_t* omega = reinterpret_cast<uint32_t*>(s->dp + L.p_omega);
  cf* g_s = reinterpret_cast<cf*>(s->dw + L.w_gs);
  const int comp = c.composition;
  // Algorithm 1's order and the additive composition select Omega from the gradient; the former then hands the
  // residual (entries at Omega zeroed in place, put back below) to the low-rank part
  if (comp != 1) {
    if (k > 0) {
      TG_TRY(select_omega<S>(s, d_grad, st));
      if (comp == 0) { scatter_zero_kernel<S><<<(k + 255) / 256, 256, 0, st>>>(d_grad, omega, k); TG_LAUNCH_CHECK(); }
    }
    TG_TRY(build_slab_ptr(s, st));
  }
  // ---- factor matrices ----
  // Starting factors: the leading eigenvectors of the mode-n Gram matrices of the residual (truncated SVDs of the
  // unfoldings).  With refinement sweeps and a warm start, the factors the state holds are the starting point
  // instead (the "warm restart" of the decomposition) and the full-size Gram matrices are not formed at all.
  bool restored = false;
  const bool from_stored = c.hooi_iters > 0 && c.warm_refresh && s->basis_valid;
  if (!from_stored) {
    int modes[TGRAD_MAX_NDIM];
    const bool warm = c.warm_refresh && s->basis_valid;
    auto gram_of = [&](int m) -> tgrad_status {
      uint64_t O = 1, C = 1;
      for (int q = 0; q < m; ++q) O *= c.dims[q];
      for (int q = m + 1; q < N; ++q) C *= c.dims[q];
      return launch_gram<S>(s, d_grad, (int)c.dims[m], O, C, L.gram_chunks[m], L.gram_cps[m], L.gram_splits[m],
                            reinterpret_cast<cf*>(s->dw + L.w_gram[m]), st);
    };
    for (int m = 0; m < N; ++m) modes[m] = m;
    const int nlead = N - 2;                       // the leading modes have the larger matrices
    RefreshStreams* rs = nlead > 0 ? refresh_streams() : nullptr;
    if (!rs) {
      for (int m = 0; m < N; ++m) TG_TRY(gram_of(m));
      TG_TRY(solve_modes(s, modes, N, warm, st));
    } else {
      for (int m = 0; m < nlead; ++m) TG_TRY(gram_of(m));
      std::lock_guard<std::mutex> lock(rs->mu);    // the events are shared by every state on this device
      if (cudaEventRecord(rs->fork, st) != cudaSuccess || cudaStreamWaitEvent(rs->side, rs->fork, 0) != cudaSuccess)
        return TGRAD_ERR_CUDA;
      tgrad_status r = solve_modes(s, modes, nlead, warm, rs->side);
      for (int m = nlead; m < N && r == TGRAD_OK; ++m) r = gram_of(m);
      // nothing reads the residual any more unless refinement sweeps follow: the gathered values go back into the
      // gradient now, beside the eigensolvers
      if (r == TGRAD_OK && k > 0 && comp == 0 && c.hooi_iters == 0) {
        scatter_restore_kernel<S><<<(k + 255) / 256, 256, 0, st>>>(d_grad, omega, g_s, k);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaPeekAtLastError() != cudaSuccess) r = TGRAD_ERR_CUDA;
        restored = true;
      }
      if (r == TGRAD_OK) r = solve_modes(s, modes + nlead, N - nlead, warm, st);
      // join even after an error, so that nothing is left running unordered
      if (cudaEventRecord(rs->join, rs->side) != cudaSuccess || cudaStreamWaitEvent(st, rs->join, 0) != cudaSuccess)
        return TGRAD_ERR_CUDA;
      TG_TRY(r);
    }
  }
  // Refinement (higher-order orthogonal iteration): per sweep and mode, compress the residual in every other mode
  // with the current factors and take the leading eigenvectors of the mode-n Gram matrix of the result.
  for (int it = 0; it < c.hooi_iters; ++it)
    for (int m = 0; m < N; ++m) TG_TRY(hooi_mode_update<S>(s, m, d_grad, st));
  if (k > 0 && comp == 0 && !restored) { scatter_restore_kernel<S><<<(k + 255) / 256, 256, 0, st>>>(d_grad, omega, g_s, k); TG_LAUNCH_CHECK(); }
  if (comp == 1) {
    // low rank first: R = G - P_U(G) in a buffer of its own (compression of G down to the core, reconstruction down
    // to the trailing modes, last two modes fused with the subtraction from a copy of G), Omega from R
    s->tabs_stale = true;                                    // the factors have just changed
    TailParams p = tail_params(s);
    p.k = 0; p.keep = 1;
    p.t = reinterpret_cast<cf*>(s->dw + L.w_bufa);
    TG_TRY(run_proj_tail(s, d_grad, p, st));
    cf* cur; uint64_t Cc;
    TG_TRY(compress_chain(s, 0, &cur, &Cc, st));
    const cf* tcore;
    TG_TRY(expand_chain(s, cur, 0, ((N - 2) & 1) ? 0 : 1, &tcore, st));
    void* rbuf = s->dw + L.w_rbuf;
    if (cudaMemcpyAsync(rbuf, d_grad, (size_t)L.numel * S::kBytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return TGRAD_ERR_CUDA;
    p.t = const_cast<cf*>(tcore);
    p.s_low = 1.0f; p.s_sparse = 0.f; p.decay = 1.0f;
    TG_TRY(run_back_tail(s, rbuf, p, st));
    if (k > 0) TG_TRY(select_omega<S>(s, rbuf, st));
    TG_TRY(build_slab_ptr(s, st));
  }
  s->have_subspace = true;
  s->tabs_stale = true;
  s->basis_valid = true;
  return TGRAD_OK;
}

tgrad_status do_refresh(tgrad_state* s, void* d_grad, cudaStream_t st) {
  return s->cfg.wg_dtype == TGRAD_C64    ? refresh_impl<StoreC64>(s, d_grad, st)
         : s->cfg.wg_dtype == TGRAD_C32H ? refresh_impl<StoreC32H>(s, d_grad, st)
                                         : refresh_impl<StoreC32B>(s, d_grad, st);
}

tgrad_status mode_product(bool conj_t, const cf* in, cf* out, const cf* U, uint64_t O, int M, int K, uint64_t C,
                          int r_n, int sm_count, cudaStream_t st) {
  // few output rows and slices that fit in shared memory: fp32 kernel with the whole slice in shared memory
  // (measured on 64x64x32x32x17: 44 instead of 60 us for the two compression products; not used for the
  // expansion, where the tensor-core tiles are full and it was slower)
  if (M <= 8 && (uint64_t)K * C <= 4096 && (uint64_t)M * C <= 4096 && (uint64_t)M * K <= 2048 && O >= 64 &&
      O < (1u << 30)) {
    const size_t smem = mode_small_smem(M, K, (int)C);
    const uint64_t cap = (uint64_t)sm_count * 8;
    const unsigned grid = (unsigned)(O < cap ? O : cap);
    if (conj_t) launch_chained(mode_product_small_kernel<true>, dim3(grid), dim3(MS_THREADS), smem, st, in, out, U, M, K, (int)C, r_n, (int)O);
    else launch_chained(mode_product_small_kernel<false>, dim3(grid), dim3(MS_THREADS), smem, st, in, out, U, M, K, (int)C, r_n, (int)O);
    TG_LAUNCH_CHECK();
    return TGRAD_OK;
  }
  // narrow column tiles when the wide ones would leave SMs without a block or two
  const uint64_t wide = ((C + 63) / 64) * ((M + MT_BM - 1) / MT_BM) * O;
  const int bc = (wide < (uint64_t)4 * sm_count) ? 32 : 64;
  dim3 grid((unsigned)((C + bc - 1) / bc), (unsigned)((M + MT_BM - 1) / MT_BM), (unsigned)O);
  if (bc == 64) {
    if (conj_t) launch_chained(mode_product_tc_kernel<true, 2>, dim3(grid), dim3(MT_THREADS), 0, st, in, out, U, M, K, (int)C, r_n);
    else launch_chained(mode_product_tc_kernel<false, 2>, dim3(grid), dim3(MT_THREADS), 0, st, in, out, U, M, K, (int)C, r_n);
  } else {
    if (conj_t) launch_chained(mode_product_tc_kernel<true, 1>, dim3(grid), dim3(MT_THREADS), 0, st, in, out, U, M, K, (int)C, r_n);
    else launch_chained(mode_product_tc_kernel<false, 1>, dim3(grid), dim3(MT_THREADS), 0, st, in, out, U, M, K, (int)C, r_n);
  }
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}

#define TG_MARK(i) do { if (evs) cudaEventRecord(evs[i], st); } while (0)

tgrad_status do_step(tgrad_state* s, void* d_weight, void* d_grad, cudaStream_t st) {
  const tgrad_config& c = s->cfg;
  const Layout& L = s->L;
  const int N = c.ndim;
  if (c.auto_refresh && (s->t % c.T) == 0) TG_TRY(do_refresh(s, d_grad, st));
  if (!s->have_subspace) return TGRAD_ERR_BAD_STATE;
  cudaEvent_t* evs = s->timing ? s->ev[s->timing_steps % kTimingRing] : nullptr;

  TailParams p = tail_params(s);
  p.adam = adam_scalars(c, s->t);
  p.keep = c.composition != 0;          // only Algorithm 1's order feeds the low-rank part with the sparse part's residual
  cf* bufa = reinterpret_cast<cf*>(s->dw + L.w_bufa);
  cf* core = reinterpret_cast<cf*>(s->dw + L.w_core);
  cf* n_l = reinterpret_cast<cf*>(s->dw + L.w_nl);
  const uint32_t ks = (uint32_t)c.k;
  const bool lr_first = c.composition == 1;

  // low-rank compression: trailing two modes while streaming G (with the sparse gather), then modes N-2 .. 1
  TG_MARK(0);
  p.t = bufa;
  TG_TRY(run_proj_tail(s, d_grad, p, st));
  TG_MARK(1);
  // the chain on the small tensor: compression of modes N-2 .. 2, then mode 1 + Adam + mode 1 in one
  // launch (or three when the first mode is too large for it), then reconstruction of modes 2 .. N-2
  // (the fused launch holds all of U^(1) and a 16-column block in shared memory and serialises its two products:
  //  beyond 64 M complex multiply-adds per product separate GEMM launches win even with the extra round trips)
  const bool fused = !lr_first && chain_fused(c);
  const cf* tprime;
  {
    cf* cur; uint64_t C;
    TG_TRY(compress_chain(s, fused ? 1 : 0, &cur, &C, st));
    TG_MARK(2);
    int which = ((N - 2) & 1) ? 0 : 1;          // make the last product land in the first buffer
    if (fused) {
      // here cur holds [I_1][C] with C = r_2 .. r_N
      cf* bufs[2] = {bufa, reinterpret_cast<cf*>(s->dw + L.w_bufb)};
      cf* dst = bufs[which];
      const uint32_t nblk_core = (uint32_t)((C + SW_CB - 1) / SW_CB), nblk_sparse = (ks + SW_THREADS - 1) / SW_THREADS;
      launch_chained(core_sandwich_tc_kernel, dim3(nblk_core + nblk_sparse), dim3(SW_THREADS), sandwich_tc_smem((int)c.dims[0], c.ranks[0]), st,
          cur, dst, reinterpret_cast<const cf*>(s->dp + L.p_factor[0]), core, reinterpret_cast<cf*>(s->dp + L.p_ml),
          reinterpret_cast<float*>(s->dp + L.p_vl), n_l, (int)c.dims[0], c.ranks[0], (int)C, p.g_s, p.m_s, p.v_s, p.n_s, ks,
          nblk_core, p.adam);
      TG_LAUNCH_CHECK();
      which ^= 1;
      TG_MARK(3);
      TG_TRY(expand_chain(s, dst, 1, which, &tprime, st));
    } else {
      if (lr_first && ks > 0) {
        // the sparse values are those of G - P_U(G): rebuild the low-rank approximation from the core down to the
        // trailing two modes and subtract its entries at Omega from the gathered ones
        const cf* tcore;
        TG_TRY(expand_chain(s, core, 0, which, &tcore, st));
        lowrank_at_omega_kernel<<<(ks + 127) / 128, 128, 0, st>>>(p.g_s, p.omega, ks, tcore, p.Ua, p.Ub, p.A, p.B, p.ra, p.rb, p.E);
        TG_LAUNCH_CHECK();
      }
      launch_chained(adam_kernel, dim3((unsigned)((L.P + ks + 255) / 256)), dim3(256), 0, st,
          core, reinterpret_cast<cf*>(s->dp + L.p_ml), reinterpret_cast<float*>(s->dp + L.p_vl), n_l, (uint32_t)L.P,
          p.g_s, p.m_s, p.v_s, p.n_s, ks, p.adam);
      TG_LAUNCH_CHECK();
      TG_MARK(3);
      TG_TRY(expand_chain(s, n_l, 0, which, &tprime, st));
    }
  }
  TG_MARK(4);
  p.t = const_cast<cf*>(tprime);
  TG_TRY(run_back_tail(s, d_weight, p, st));
  TG_MARK(5);
  if (s->timing) s->timing_steps++;
  s->t += 1;
  return TGRAD_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Side streams of the batched step, one set per device, created at the first batched call on that device and kept
// for the life of the process.
constexpr int kBatchStreams = 4, kBatchDevices = 64;
struct BatchStreams {
  std::mutex mu;
  bool ready = false;
  cudaStream_t side[kBatchStreams];
  cudaEvent_t fork, join[kBatchStreams];
};
BatchStreams g_batch[kBatchDevices];
BatchStreams* batch_streams() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kBatchDevices) return nullptr;
  BatchStreams* b = &g_batch[dev];
  std::lock_guard<std::mutex> lock(b->mu);
  if (!b->ready) {
    bool ok = cudaEventCreateWithFlags(&b->fork, cudaEventDisableTiming) == cudaSuccess;
    for (int j = 0; ok && j < kBatchStreams; ++j)
      ok = cudaStreamCreateWithFlags(&b->side[j], cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&b->join[j], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) return nullptr;          // fall back to the caller's stream alone
    b->ready = true;
  }
  return b;
}

}  // namespace

extern "C" {

tgrad_status tgrad_state_bytes(const tgrad_config* cfg, size_t* persistent_bytes, size_t* workspace_bytes) {
  if (!persistent_bytes || !workspace_bytes) return TGRAD_ERR_INVALID_ARG;
  Layout L;
  tgrad_config ic; int map[TGRAD_MAX_NDIM];
  tgrad_status s = internal_config(cfg, ic, map);
  if (s != TGRAD_OK) return s;
  // The split-K plan of the Gram kernels (part of the workspace size) is made for 148 SMs whatever the device:
  // the sizes a configuration needs are then the same on every machine, and the kernels only need a plan, not
  // the best one.
  s = compute_layout(&ic, L, 148);
  if (s != TGRAD_OK) return s;
  *persistent_bytes = L.p_total;
  *workspace_bytes = L.w_total;
  return TGRAD_OK;
}

tgrad_status tgrad_init_state(const tgrad_config* cfg, void* d_persistent, size_t persistent_bytes, void* d_workspace,
                              size_t workspace_bytes, void* cuda_stream, tgrad_state** out) {
  if (!out) return TGRAD_ERR_INVALID_ARG;
  *out = nullptr;
  Layout L;
  tgrad_config ic; int map[TGRAD_MAX_NDIM];
  tgrad_status s = internal_config(cfg, ic, map);
  if (s != TGRAD_OK) return s;
  s = compute_layout(&ic, L, 148);
  if (s != TGRAD_OK) return s;
  cfg = &ic;
  if (!d_persistent || !d_workspace) return TGRAD_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_persistent) & 255) || (reinterpret_cast<uintptr_t>(d_workspace) & 255))
    return TGRAD_ERR_INVALID_ARG;
  if (persistent_bytes < L.p_total || workspace_bytes < L.w_total) return TGRAD_ERR_BUFFER_TOO_SMALL;
  tgrad_state* st = new (std::nothrow) tgrad_state;
  if (!st) return TGRAD_ERR_INVALID_ARG;
  memset(st, 0, sizeof(*st));
  st->cfg = *cfg; st->L = L;
  st->ext_ndim = (ic.ndim == 3 && map[1] == 2) ? 2 : ic.ndim;
  for (int n = 0; n < TGRAD_MAX_NDIM; ++n) st->mode_map[n] = map[n];
  st->dp = static_cast<char*>(d_persistent); st->dw = static_cast<char*>(d_workspace);
  st->t = 0; st->have_subspace = false; st->tabs_stale = true; st->basis_valid = false;
  int dev = 0, sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { delete st; return TGRAD_ERR_CUDA; }
  st->sm_count = sm;
  s = plan_tail(st);
  if (s != TGRAD_OK) { delete st; return s; }
  {
    bool ok = true;
#define TG_GRAM_ATTR(S_, SPLIT_, FULL_)                                                                       \
  ok = ok && cudaFuncSetAttribute(gram_partial_kernel<S_, SPLIT_, FULL_>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                  (int)GR_SMEM) == cudaSuccess
    TG_GRAM_ATTR(StoreC64, false, false); TG_GRAM_ATTR(StoreC64, false, true);
    TG_GRAM_ATTR(StoreC64, true, false); TG_GRAM_ATTR(StoreC64, true, true);
    TG_GRAM_ATTR(StoreC32H, false, false); TG_GRAM_ATTR(StoreC32H, false, true);
    TG_GRAM_ATTR(StoreC32H, true, false); TG_GRAM_ATTR(StoreC32H, true, true);
    TG_GRAM_ATTR(StoreC32B, false, false); TG_GRAM_ATTR(StoreC32B, false, true);
    TG_GRAM_ATTR(StoreC32B, true, false); TG_GRAM_ATTR(StoreC32B, true, true);
#undef TG_GRAM_ATTR
    ok = ok && cudaFuncSetAttribute(gram_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemMax - 1024)) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(gram_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemMax - 1024)) == cudaSuccess;
    ok = ok && cudaFuncSetAttribute(gram_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kSmemMax - 1024)) == cudaSuccess;
    if (!ok) { delete st; return TGRAD_ERR_CUDA; }
  }
  if (cfg->dims[0] <= SW_MAX_I && cfg->ranks[0] <= SW_MAX_R &&
      cudaFuncSetAttribute(core_sandwich_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)sandwich_tc_smem(SW_MAX_I, SW_MAX_R)) != cudaSuccess) { delete st; return TGRAD_ERR_CUDA; }
  if (cudaFuncSetAttribute(subspace_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMax) != cudaSuccess) {
    delete st; return TGRAD_ERR_CUDA;
  }
  if (cudaFuncSetAttribute(jacobi_sweeps_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)jac_sweeps_smem(JAC_SMEM_MAX_N)) != cudaSuccess) { delete st; return TGRAD_ERR_CUDA; }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // Algorithm 1 initialisation: zero moments (and flags, Omega, factors for determinism)
  if (cudaMemsetAsync(d_persistent, 0, L.p_total, stream) != cudaSuccess) { delete st; return TGRAD_ERR_CUDA; }
  *out = st;
  return TGRAD_OK;
}

tgrad_status tgrad_step(tgrad_state* st, void* d_weight, void* d_grad, void* cuda_stream) {
  if (!st || !d_weight || !d_grad) return TGRAD_ERR_INVALID_ARG;
  if (!aligned16(d_weight) || !aligned16(d_grad)) return TGRAD_ERR_INVALID_ARG;
  return do_step(st, d_weight, d_grad, static_cast<cudaStream_t>(cuda_stream));
}

tgrad_status tgrad_refresh_subspace(tgrad_state* st, void* d_grad, void* cuda_stream) {
  if (!st || !d_grad) return TGRAD_ERR_INVALID_ARG;
  if (!aligned16(d_grad)) return TGRAD_ERR_INVALID_ARG;
  return do_refresh(st, d_grad, static_cast<cudaStream_t>(cuda_stream));
}

tgrad_status tgrad_step_batched(tgrad_state* const* states, void* const* d_weights, void* const* d_grads,
                                int32_t n_tensors, void* cuda_stream) {
  if (n_tensors < 0 || (n_tensors > 0 && (!states || !d_weights || !d_grads))) return TGRAD_ERR_INVALID_ARG;
  for (int i = 0; i < n_tensors; ++i) {
    if (!states[i] || !d_weights[i] || !d_grads[i]) return TGRAD_ERR_INVALID_ARG;
    if (!aligned16(d_weights[i]) || !aligned16(d_grads[i])) return TGRAD_ERR_INVALID_ARG;
    if (!states[i]->have_subspace && !(states[i]->cfg.auto_refresh && states[i]->t % states[i]->cfg.T == 0))
      return TGRAD_ERR_BAD_STATE;
  }
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  // The chains of small tensors are bound by launch and dependency latency, not by the GPU, and the tensors are
  // independent: fork them onto the library's side streams and join them back into the caller's stream.  Work
  // enqueued on the caller's stream before this call happens before all of it, work enqueued after it happens after.
  BatchStreams* bs = (n_tensors > 1) ? batch_streams() : nullptr;
  if (!bs) {
    for (int i = 0; i < n_tensors; ++i) TG_TRY(do_step(states[i], d_weights[i], d_grads[i], user));
    return TGRAD_OK;
  }
  std::lock_guard<std::mutex> lock(bs->mu);
  if (cudaEventRecord(bs->fork, user) != cudaSuccess) return TGRAD_ERR_CUDA;
  const int lanes = n_tensors < kBatchStreams ? n_tensors : kBatchStreams;
  for (int j = 0; j < lanes; ++j)
    if (cudaStreamWaitEvent(bs->side[j], bs->fork, 0) != cudaSuccess) return TGRAD_ERR_CUDA;
  tgrad_status result = TGRAD_OK;
  for (int i = 0; i < n_tensors && result == TGRAD_OK; ++i) result = do_step(states[i], d_weights[i], d_grads[i], bs->side[i % lanes]);
  for (int j = 0; j < lanes; ++j) {           // join even after an error, so that nothing is left running unordered
    if (cudaEventRecord(bs->join[j], bs->side[j]) != cudaSuccess || cudaStreamWaitEvent(user, bs->join[j], 0) != cudaSuccess)
      return TGRAD_ERR_CUDA;
  }
  return result;
}

tgrad_status tgrad_refresh_subspace_batched(tgrad_state* const* states, void* const* d_grads, int32_t n_tensors,
                                            void* cuda_stream) {
  if (n_tensors < 0 || (n_tensors > 0 && (!states || !d_grads))) return TGRAD_ERR_INVALID_ARG;
  for (int i = 0; i < n_tensors; ++i)
    if (!states[i] || !d_grads[i] || !aligned16(d_grads[i])) return TGRAD_ERR_INVALID_ARG;
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  // as in the batched step: the tensors' refreshes are independent, so they are forked onto the side streams
  BatchStreams* bs = (n_tensors > 1) ? batch_streams() : nullptr;
  if (!bs) {
    for (int i = 0; i < n_tensors; ++i) TG_TRY(do_refresh(states[i], d_grads[i], user));
    return TGRAD_OK;
  }
  std::lock_guard<std::mutex> lock(bs->mu);
  if (cudaEventRecord(bs->fork, user) != cudaSuccess) return TGRAD_ERR_CUDA;
  const int lanes = n_tensors < kBatchStreams ? n_tensors : kBatchStreams;
  for (int j = 0; j < lanes; ++j)
    if (cudaStreamWaitEvent(bs->side[j], bs->fork, 0) != cudaSuccess) return TGRAD_ERR_CUDA;
  tgrad_status result = TGRAD_OK;
  for (int i = 0; i < n_tensors && result == TGRAD_OK; ++i) result = do_refresh(states[i], d_grads[i], bs->side[i % lanes]);
  for (int j = 0; j < lanes; ++j) {           // join even after an error, so that nothing is left running unordered
    if (cudaEventRecord(bs->join[j], bs->side[j]) != cudaSuccess || cudaStreamWaitEvent(user, bs->join[j], 0) != cudaSuccess)
      return TGRAD_ERR_CUDA;
  }
  return result;
}

tgrad_status tgrad_query_status(tgrad_state* st, void* cuda_stream, int32_t* sticky_flags, int64_t* t, int32_t* sweeps) {
  if (!st) return TGRAD_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int host[1 + TGRAD_MAX_NDIM];
  if (cudaMemcpyAsync(host, st->dp + st->L.p_flags, sizeof(host), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return TGRAD_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (sticky_flags) *sticky_flags = host[0];
  if (t) *t = st->t;
  if (sweeps) for (int n = 0; n < st->ext_ndim; ++n) sweeps[n] = host[1 + st->mode_map[n]];
  return TGRAD_OK;
}

static tgrad_status locate(tgrad_state* st, int32_t what, bool for_import, char** ptr, size_t* bytes) {
  const tgrad_config& c = st->cfg; const Layout& L = st->L;
  const size_t k = (size_t)c.k, P = (size_t)L.P;
  switch (what) {
    case TGRAD_WHAT_OMEGA: *ptr = st->dp + L.p_omega; *bytes = k * 4; return TGRAD_OK;
    case TGRAD_WHAT_M_L: *ptr = st->dp + L.p_ml; *bytes = P * 8; return TGRAD_OK;
    case TGRAD_WHAT_V_L: *ptr = st->dp + L.p_vl; *bytes = P * 4; return TGRAD_OK;
    case TGRAD_WHAT_M_S: *ptr = st->dp + L.p_ms; *bytes = k * 8; return TGRAD_OK;
    case TGRAD_WHAT_V_S: *ptr = st->dp + L.p_vs; *bytes = k * 4; return TGRAD_OK;
    default: break;
  }
  if (what >= TGRAD_WHAT_FACTOR_BASE && what < TGRAD_WHAT_FACTOR_BASE + st->ext_ndim) {
    int n = st->mode_map[what - TGRAD_WHAT_FACTOR_BASE];
    *ptr = st->dp + L.p_factor[n]; *bytes = (size_t)c.dims[n] * c.ranks[n] * 8; return TGRAD_OK;
  }
  if (for_import) return TGRAD_ERR_INVALID_ARG;
  switch (what) {
    case TGRAD_WHAT_CORE: *ptr = st->dw + L.w_core; *bytes = P * 8; return TGRAD_OK;
    case TGRAD_WHAT_N_L: *ptr = st->dw + L.w_nl; *bytes = P * 8; return TGRAD_OK;
    case TGRAD_WHAT_N_S: *ptr = st->dw + L.w_ns; *bytes = k * 8; return TGRAD_OK;
    default: break;
  }
  if (what >= TGRAD_WHAT_GRAM_BASE && what < TGRAD_WHAT_GRAM_BASE + st->ext_ndim) {
    int n = st->mode_map[what - TGRAD_WHAT_GRAM_BASE];
    *ptr = st->dw + L.w_gram[n]; *bytes = (size_t)c.dims[n] * c.dims[n] * 8; return TGRAD_OK;
  }
  return TGRAD_ERR_INVALID_ARG;
}

tgrad_status tgrad_export_state(tgrad_state* st, int32_t what, void* host_dst, size_t bytes, void* cuda_stream) {
  if (!st || (!host_dst && bytes)) return TGRAD_ERR_INVALID_ARG;
  char* p; size_t nb;
  tgrad_status s = locate(st, what, false, &p, &nb);
  if (s != TGRAD_OK) return s;
  if (bytes != nb) return TGRAD_ERR_BUFFER_TOO_SMALL;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (nb && cudaMemcpyAsync(host_dst, p, nb, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  return TGRAD_OK;
}

tgrad_status tgrad_import_state(tgrad_state* st, int32_t what, const void* host_src, size_t bytes, void* cuda_stream) {
  if (!st || (!host_src && bytes)) return TGRAD_ERR_INVALID_ARG;
  char* p; size_t nb;
  tgrad_status s = locate(st, what, true, &p, &nb);
  if (s != TGRAD_OK) return s;
  if (bytes != nb) return TGRAD_ERR_BUFFER_TOO_SMALL;
  if (what == TGRAD_WHAT_OMEGA) {   // Omega must be strictly ascending and in range
    const uint32_t* om = static_cast<const uint32_t*>(host_src);
    const size_t k = (size_t)st->cfg.k;
    for (size_t j = 0; j < k; ++j) {
      if ((uint64_t)om[j] >= st->L.numel) return TGRAD_ERR_INVALID_ARG;
      if (j && om[j] <= om[j - 1]) return TGRAD_ERR_INVALID_ARG;
    }
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (nb && cudaMemcpyAsync(p, host_src, nb, cudaMemcpyHostToDevice, stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (what == TGRAD_WHAT_OMEGA) {
    tgrad_status r = build_slab_ptr(st, stream);
    if (r != TGRAD_OK) return r;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  }
  if (what == TGRAD_WHAT_OMEGA || what >= TGRAD_WHAT_FACTOR_BASE) st->have_subspace = true;
  if (what >= TGRAD_WHAT_FACTOR_BASE) { st->tabs_stale = true; st->basis_valid = true; }
  return TGRAD_OK;
}

tgrad_status tgrad_diagnostics(tgrad_state* st, const void* d_grad, void* cuda_stream, double* out) {
  if (!st || !d_grad || !out) return TGRAD_ERR_INVALID_ARG;
  if (!aligned16(d_grad)) return TGRAD_ERR_INVALID_ARG;
  if (!st->have_subspace || st->t < 1) return TGRAD_ERR_BAD_STATE;
  const tgrad_config& c = st->cfg; const Layout& L = st->L;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  double* acc = reinterpret_cast<double*>(st->dw + L.w_diag);
  if (cudaMemsetAsync(acc, 0, 8 * sizeof(double), stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  const unsigned gsz = (unsigned)(st->sm_count * 8);
  if (c.wg_dtype == TGRAD_C64) diag_sumsq_kernel<StoreC64><<<gsz, 256, 0, stream>>>(d_grad, L.numel, acc + 0);
  else if (c.wg_dtype == TGRAD_C32H) diag_sumsq_kernel<StoreC32H><<<gsz, 256, 0, stream>>>(d_grad, L.numel, acc + 0);
  else diag_sumsq_kernel<StoreC32B><<<gsz, 256, 0, stream>>>(d_grad, L.numel, acc + 0);
  TG_LAUNCH_CHECK();
  if (c.k > 0) { diag_sumsq_kernel<StoreC64><<<64, 256, 0, stream>>>(st->dw + L.w_gs, (uint64_t)c.k, acc + 1); TG_LAUNCH_CHECK(); }
  diag_sumsq_kernel<StoreC64><<<64, 256, 0, stream>>>(st->dw + L.w_core, L.P, acc + 2); TG_LAUNCH_CHECK();
  for (int n = 0; n < c.ndim; ++n) {
    const int r = c.ranks[n];
    diag_ortho_kernel<<<(r * r + 127) / 128, 128, 0, stream>>>(reinterpret_cast<const cf*>(st->dp + L.p_factor[n]), (int)c.dims[n], r,
                                                              reinterpret_cast<unsigned int*>(acc + 3));
    TG_LAUNCH_CHECK();
  }
  double host[4];
  if (cudaMemcpyAsync(host, acc, sizeof(host), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return TGRAD_ERR_CUDA;
  const double g2 = host[0], s2 = host[1], l2 = host[2];
  unsigned int bits; memcpy(&bits, &host[3], sizeof(bits));
  float defect; memcpy(&defect, &bits, sizeof(defect));
  // what the low-rank part was given: the residual of the sparse part in Algorithm 1's order (the sparse values were
  // gathered from the gradient itself there), the gradient otherwise
  const double x2 = (c.composition == 0) ? (g2 - s2 > 0 ? g2 - s2 : 0.0) : g2;
  const double gn = std::sqrt(g2);
  out[0] = gn;
  out[1] = gn > 0 ? std::sqrt(s2) / gn : 0.0;
  out[2] = gn > 0 ? std::sqrt(x2 - l2 > 0 ? x2 - l2 : 0.0) / gn : 0.0;
  out[3] = (double)defect;
  return TGRAD_OK;
}

tgrad_status tgrad_set_step(tgrad_state* st, int64_t t) {
  if (!st || t < 0) return TGRAD_ERR_INVALID_ARG;
  st->t = t;
  return TGRAD_OK;
}

tgrad_status tgrad_set_stage_timing(tgrad_state* st, int32_t enable) {
  if (!st) return TGRAD_ERR_INVALID_ARG;
  if (enable && !st->ev[0][0]) {
    for (int i = 0; i < kTimingRing; ++i)
      for (int j = 0; j <= kStages; ++j)
        if (cudaEventCreate(&st->ev[i][j]) != cudaSuccess) return TGRAD_ERR_CUDA;
  }
  st->timing = enable != 0;
  st->timing_steps = 0;
  return TGRAD_OK;
}

tgrad_status tgrad_get_stage_times(tgrad_state* st, void* cuda_stream, float* ms_sum, int32_t* n_steps) {
  if (!st || !ms_sum || !n_steps) return TGRAD_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return TGRAD_ERR_CUDA;
  int n = st->timing_steps < kTimingRing ? st->timing_steps : kTimingRing;
  for (int j = 0; j < kStages; ++j) ms_sum[j] = 0.f;
  for (int i = 0; i < n; ++i)
    for (int j = 0; j < kStages; ++j) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, st->ev[i][j], st->ev[i][j + 1]) != cudaSuccess) return TGRAD_ERR_CUDA;
      ms_sum[j] += ms;
    }
  *n_steps = n;
  st->timing_steps = 0;
  return TGRAD_OK;
}

tgrad_status tgrad_destroy_state(tgrad_state* st) {
  if (!st) return TGRAD_ERR_INVALID_ARG;
  if (st->ev[0][0])
    for (int i = 0; i < kTimingRing; ++i)
      for (int j = 0; j <= kStages; ++j)
        if (st->ev[i][j]) cudaEventDestroy(st->ev[i][j]);
  delete st;
  return TGRAD_OK;
}

const char* tgrad_status_string(tgrad_status s) {
  switch (s) {
    case TGRAD_OK: return "ok";
    case TGRAD_ERR_INVALID_ARG: return "invalid argument";
    case TGRAD_ERR_UNSUPPORTED: return "unsupported configuration";
    case TGRAD_ERR_BUFFER_TOO_SMALL: return "buffer size mismatch";
    case TGRAD_ERR_CUDA: return "CUDA error";
    case TGRAD_ERR_NO_CONVERGE: return "eigensolver did not converge";
    case TGRAD_ERR_NONFINITE: return "non-finite gradient";
    case TGRAD_ERR_BAD_STATE: return "state has no subspace yet";
    case TGRAD_ERR_TOO_LARGE: return "input exceeds the built-in scratch of the allocation-free entry point";
    default: return "unknown status";
  }
}

int64_t tgrad_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Allocation-free top-k selection.  Its scratch is a fixed array in the device image; the name
// below is usable as an address in device code only -- host code asks the runtime for the
// device address (once per device) and hands that to the kernels.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr uint64_t kNaMaxNumel = (uint64_t)TGRAD_NOALLOC_MAX_NUMEL;
constexpr uint32_t kNaMaxBlocks = (uint32_t)(kNaMaxNumel / kChunk);
struct NoAllocScratch {
  SelState sel;
  int flags[4];
  uint32_t hist[3 * kSelMaxBins];
  uint32_t blk[2 * kNaMaxBlocks];
};
constexpr int kNaMaxDevices = 64;
std::mutex g_na_mu;
void* g_na_addr[kNaMaxDevices];
int g_na_sm[kNaMaxDevices];
}  // namespace

static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

namespace {
// Device address of the scratch array on the current device; looked up on the first call per device.
tgrad_status noalloc_scratch(NoAllocScratch** out, int* sm_count) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TGRAD_ERR_CUDA;
  if (dev < 0 || dev >= kNaMaxDevices) return TGRAD_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_na_mu);
  if (!g_na_addr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return TGRAD_ERR_CUDA;
    int sm = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm < 1) return TGRAD_ERR_CUDA;
    g_na_addr[dev] = ptr; g_na_sm[dev] = sm;
  }
  *out = static_cast<NoAllocScratch*>(g_na_addr[dev]);
  *sm_count = g_na_sm[dev];
  return TGRAD_OK;
}

template <class S>
tgrad_status select_noalloc_impl(const void* d_grad, uint32_t n, uint32_t k, uint32_t* d_omega, cf* d_values,
                                 NoAllocScratch* sc, int sm, cudaStream_t st) {
  const uint32_t nblk = (n + kChunk - 1) / kChunk;
  SelKey kp; kp.seed_lo = kp.seed_hi = kp.epoch = 0u; kp.strategy = 0;     // magnitude top-k
  uint32_t* blk_gt = sc->blk;
  uint32_t* blk_eq = sc->blk + nblk;
  // the histograms and the flag word must start at zero; everything else is overwritten before it is read
  if (cudaMemsetAsync(sc->flags, 0, sizeof(sc->flags) + sizeof(sc->hist), st) != cudaSuccess) return TGRAD_ERR_CUDA;
  sel_init_kernel<<<1, 1, 0, st>>>(&sc->sel, k, 0u); TG_LAUNCH_CHECK();
  const uint64_t want = ((uint64_t)n + 511) / 512;
  const int hgrid = (int)(want < (uint64_t)sm * 8 ? want : (uint64_t)sm * 8);
  for (int pass = 0; pass < 3; ++pass) {
    sel_hist_kernel<S, true><<<hgrid, 512, 0, st>>>(d_grad, n, pass, &sc->sel, sc->hist + pass * kSelMaxBins, sc->flags, kp);
    TG_LAUNCH_CHECK();
    sel_pick_kernel<<<1, 1024, 0, st>>>(sc->hist + pass * kSelMaxBins, pass, &sc->sel); TG_LAUNCH_CHECK();
  }
  sel_count_kernel<S, true><<<nblk, kChunkThreads, 0, st>>>(d_grad, n, &sc->sel, blk_gt, blk_eq, kp); TG_LAUNCH_CHECK();
  sel_scan_kernel<<<1, 1024, 0, st>>>(blk_gt, blk_eq, nblk); TG_LAUNCH_CHECK();
  sel_compact_kernel<S, true><<<nblk, kChunkThreads, 0, st>>>(d_grad, n, &sc->sel, blk_gt, blk_eq, d_omega, d_values, k, kp);
  TG_LAUNCH_CHECK();
  return TGRAD_OK;
}
}  // namespace

extern "C" tgrad_status tgrad_select_topk_noalloc(const void* d_grad, int64_t numel, int64_t k, int32_t wg_dtype,
                                                  uint32_t* d_omega, void* d_values, void* cuda_stream) {
  if (numel < 1 || k < 0 || k > numel) return TGRAD_ERR_INVALID_ARG;
  if (wg_dtype != TGRAD_C64 && wg_dtype != TGRAD_C32H && wg_dtype != TGRAD_C32B) return TGRAD_ERR_INVALID_ARG;
  if ((uint64_t)numel > kNaMaxNumel) return TGRAD_ERR_TOO_LARGE;
  if (!d_grad || (k > 0 && (!d_omega || !d_values))) return TGRAD_ERR_INVALID_ARG;
  // the kernels read the gradient with vector loads and write index / value pairs: same rule as the other calls
  if (!aligned16(d_grad) || (k > 0 && (!aligned16(d_omega) || !aligned16(d_values)))) return TGRAD_ERR_INVALID_ARG;
  if (k == 0) return TGRAD_OK;
  NoAllocScratch* sc = nullptr;
  int sm = 0;
  tgrad_status r = noalloc_scratch(&sc, &sm);
  if (r != TGRAD_OK) return r;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (wg_dtype == TGRAD_C64)
    return select_noalloc_impl<StoreC64>(d_grad, (uint32_t)numel, (uint32_t)k, d_omega, static_cast<cf*>(d_values), sc, sm, st);
  if (wg_dtype == TGRAD_C32H)
    return select_noalloc_impl<StoreC32H>(d_grad, (uint32_t)numel, (uint32_t)k, d_omega, static_cast<cf*>(d_values), sc, sm, st);
  return select_noalloc_impl<StoreC32B>(d_grad, (uint32_t)numel, (uint32_t)k, d_omega, static_cast<cf*>(d_values), sc, sm, st);
}
