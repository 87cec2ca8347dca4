// grass_project_grad: host side (argument checks, tiling plan, TMA descriptors,
// launches).  The kernels are in project_tc.cuh (bf16, tcgen05) and
// project_simt.cuh (fp32).
#include <cudaTypedefs.h>

#include "common.cuh"
#include "project_simt.cuh"
#include "project_tc.cuh"

namespace grass {
namespace {

constexpr int kSmCount = 148;

// How the selected dY columns reach the GEMM (values of grass_project_opts_t::gather; 0 in a
// plan means the operand is dY itself, i.e. the dense gradient).
constexpr int kOptAuto = 0, kOptPrepass = 1, kOptCta = 2, kOptCoop = 3;

struct PlanOpts {
  int gather = kOptAuto;   // kOpt*
  int mb = 0;              // n-blocks of 128 columns per CTA: 0 = cost model, else 1, 2 or 4 if it fits
  int pair = 0;            // 0 = cost model, 1 = single CTAs only, 2 = CTA pairs wherever the shape allows
  int split = 0;           // token slices: 0 = cost model
  int gather_warps = 0;    // cooperative gather: warps per CTA that gather (0 = default)
};

PlanOpts to_plan_opts(const grass_project_opts_t* o) {
  PlanOpts po;
  if (o != nullptr) {
    po.gather = o->gather;
    po.mb = o->n_blocks_per_cta;
    po.pair = o->cta_pair;
    po.split = o->token_slices;
    po.gather_warps = o->gather_warps;
  }
  return po;
}
bool opts_ok(const grass_project_opts_t* o) {
  return o == nullptr ||
         (o->gather >= kOptAuto && o->gather <= kOptCoop &&
          (o->n_blocks_per_cta == 0 || o->n_blocks_per_cta == 1 || o->n_blocks_per_cta == 2 ||
           o->n_blocks_per_cta == 4) &&
          o->cta_pair >= 0 && o->cta_pair <= 2 && o->token_slices >= 0 &&
          o->gather_warps >= 0 && o->gather_warps <= 8);
}

struct TcPlan {
  int gather;     // 0: operand read from dY as it is; else kOptPrepass / kOptCta / kOptCoop
  int kb_unit;    // token slices start on multiples of this many token blocks
  size_t ctrl_bytes;   // cooperative gather: queue head and per-chunk counters
  int r_pad;      // r_blocks * r_cta: width of the gathered operand
  int r_cta, r_blocks;
  int MB, n_blocks;   // n_blocks = CTAs along n (an even number when pair)
  bool pair;          // two CTAs share each MMA (cta_group::2)
  int k_blocks, stages, bk;   // bk: tokens per pipeline stage
  int split_k, s_long;        // token slices; the first s_long are long, the rest short
  int unit_begin[kTcMaxSlices + 1];   // slice z = units [unit_begin[z], unit_begin[z + 1])
  size_t smem_bytes;
  long long ld_part;        // pitch of a split-K partial, elements
  size_t ag_bytes, part_bytes;
};

// How the selected columns get to the GEMM for a given tile shape.  In-CTA gather: the GEMM's
// own warps pick the columns out of dY into shared memory.  It pays when a tile holds at most
// 128 rows (the load unit keeps up), at most two CTAs (pairs) share a token slice (each gathers
// for itself) and the picks are dense enough that a 32-lane load spans at most 6 cache lines
// (12 r >= m); measured on the 60M q,k,v,o group (m = 512, r = 128): step 253 -> 274 TFLOP/s,
// while at m = 2048, r = 128 the sparser pick made the in-kernel loads the bottleneck.
// Everything else: cooperative gather (all CTAs share one pass over dY, overlapped with the
// MMAs); the stand-alone pre-pass remains selectable.
int choose_gather(bool has_idx, const PlanOpts& opts, int r_cta, int tiles_x, int64_t m, int r) {
  if (!has_idx) return 0;
  const bool cta_ok = r_cta <= 128;
  if (opts.gather == kOptCta && cta_ok) return kOptCta;
  if (opts.gather == kOptPrepass) return kOptPrepass;
  if (opts.gather == kOptCoop) return kOptCoop;
  if (opts.gather == kOptAuto && cta_ok && tiles_x <= 2 && static_cast<int64_t>(r) * 12 >= m)
    return kOptCta;
  // Few selected rows (r <= 128): the GEMM is a pure HBM stream of X and the gather is as large
  // as the GEMM itself; as two kernels the gather of one layer overlaps the GEMM of another
  // stream's layer, which measured better than one kernel doing both (1B shapes, r = 64 / 128:
  // 98 / 116 us per layer-step against 107 / 128).
  if (opts.gather == kOptAuto && cta_ok) return kOptPrepass;
  return kOptCoop;
}

// Choose the CTA tile and the token slices.  Cost model in SM clocks.  A worker (a CTA, or a
// CTA pair) needs `c` clocks per unit of tokens and `f` clocks per tile (pipeline fill,
// epilogue).  With N = tiles-per-slice x slices tiles on W workers the time is that of the
// busiest worker; equal slices leave the last wave partly empty whenever W does not divide N.
// So besides s_long equal slices the search tries up to three extra SHORT slices: the
// R = N_long mod W workers that receive one long tile more than the rest are then finished,
// and the other W - R workers share the short tiles; the lengths (x units long, y units short)
// are set so that both kinds of worker finish together:
//     x c + f = ns (y c + f),  s_long x + s_short y = U,  ns = ceil(N_short / (W - R)).
// The operands reach the SMs from L2 (every CTA fetches its own tiles): the X tile of an n-block
// once per row block and the gathered operand once per n-tile.  On the LLaMA-7B r = 1024 shapes
// this traffic (about 8.6 TB/s), not the number of busy SMs, bounds the kernel: the same 187 us
// with 128 or with all 148 SMs at work.  Split-K partials cost their HBM write plus re-read.  Smaller n-tiles (MB) make more,
// smaller CTAs, which cuts partial traffic when the output is tiny; larger ones cut the number
// of times the gathered operand is re-read.  The result depends only on the arguments.
TcPlan make_plan(int64_t T, int64_t m, int64_t n, int r, bool has_idx, const PlanOpts& opts,
                 bool single_split = false, int groups = 1) {
  TcPlan p;
  const int r64 = static_cast<int>(round_up(static_cast<size_t>(r), 64));
  p.r_blocks = (r64 + 511) / 512;
  p.r_cta = static_cast<int>(round_up(static_cast<size_t>((r64 + p.r_blocks - 1) / p.r_blocks), 64));
  p.r_pad = p.r_cta * p.r_blocks;
  int mb_max = 512 / p.r_cta;
  mb_max = mb_max >= 4 ? 4 : (mb_max >= 2 ? 2 : 1);
  while (mb_max > 1 && static_cast<int64_t>(mb_max / 2) * 128 >= n) mb_max /= 2;  // not past n

  const double hbm_bytes_per_clk = 6.5e12 / 1.7e9;  // whole chip, per SM clock
  double best = 1e300;
  p.MB = 1;
  p.pair = false;
  p.split_k = p.s_long = 1;
  int best_x = 0;            // units per long slice (0: equal slices)
  const bool can_pair = (p.r_cta % 128) == 0 && opts.pair != 1;
  for (int mb = mb_max; mb >= 1; mb /= 2) {
    if (opts.mb > 0 && opts.mb <= mb_max && mb != opts.mb) continue;
    for (int pair = can_pair ? 1 : 0; pair >= 0; --pair) {
      if (pair && n <= static_cast<int64_t>(mb) * 128) continue;  // nothing for the second CTA
      if (!pair && opts.pair == 2 && can_pair && n > static_cast<int64_t>(mb) * 128) continue;
      const int cta_cols = mb * 128 * (pair ? 2 : 1);
      const int tiles_x = static_cast<int>((n + cta_cols - 1) / cta_cols);
      const int64_t n_out = static_cast<int64_t>(tiles_x) * p.r_blocks * groups;   // tiles per slice
      const int W = pair ? kSmCount / 2 : kSmCount;
      const int a_slabs = pair ? p.r_cta / 128 : p.r_cta / 64;
      const int bk = tc_bk(mb, a_slabs);
      const int gather = choose_gather(has_idx, opts, p.r_cta, tiles_x, m, r);
      const int unit_tokens = gather == kOptCoop ? kCoopChunk : bk;
      const int U = static_cast<int>((T + unit_tokens - 1) / unit_tokens);
      // clocks per 32 tokens of one CTA: tensor time, or (single CTA) the shared-memory ceiling;
      // never less than 256 (a CTA cannot stream its operands faster)
      double c = static_cast<double>(mb) * p.r_cta;
      if (!pair) c *= 1.4;
      if (c < 256.0) c = 256.0;
      c *= unit_tokens / 32.0;
      const double f = 3000.0 + mb * 128.0 * p.r_cta * 4.0 / 128.0;   // pipeline fill, accumulator drain
      // L2 -> SM bytes of the whole launch (per CTA and 32 tokens: (columns + rows) x 64 bytes) at
      // about 8.6 TB/s.  It overlaps the MMAs only in part: half of it is charged, which is what
      // makes wider n-tiles (fewer re-reads of the gathered operand) win on the HBM-bound shapes.
      const double cta_rows = pair ? p.r_cta / 2 : p.r_cta;
      const double l2_clk = static_cast<double>(tiles_x) * p.r_blocks * groups * (pair ? 2 : 1) *
                            static_cast<double>((T + 31) / 32) * (mb * 128.0 + cta_rows) * 64.0 / 4500.0;
      const int max_s = single_split ? 1 : (U < kTcMaxSlices ? U : kTcMaxSlices);
      for (int sl = 1; sl <= max_s; ++sl) {
        if (opts.split > 0 && !single_split && sl != (opts.split < max_s ? opts.split : max_s)) continue;
        const int64_t n_long = n_out * sl;
        const int64_t F = n_long / W, R = n_long % W;
        // short slices where they were measured to pay: launches of three or more waves
        // (7B down, r = 1024: 587 -> 539 us), and the in-CTA gather, where each worker is bound
        // by its own gather warps (60M q,k,v,o: 179 -> 155 us).  With fewer waves the kernel is
        // bound by operand traffic, and the extra partials cost more than the idle SMs.
        const int max_short =
            (single_split || opts.split > 0 || R == 0 || (F < 2 && gather != kOptCta)) ? 0 : 3;
        for (int ss = 0; ss <= max_short && sl + ss <= max_s; ++ss) {
          double span;
          int x_units = 0;
          if (ss == 0) {
            span = static_cast<double>((n_long + W - 1) / W) * (((U + sl - 1) / sl) * c + f);
          } else {
            const int64_t ns = (n_out * ss + (W - R) - 1) / (W - R);
            const double x = (U + ss * (f / c) * (1.0 - 1.0 / ns)) / (sl + static_cast<double>(ss) / ns);
            span = 1e300;
            for (int cand = static_cast<int>(x); cand <= static_cast<int>(x) + 1; ++cand) {
              const int y_total = U - sl * cand;
              if (cand < 1 || y_total < ss) continue;
              const int y_max = (y_total + ss - 1) / ss;
              const double a = (F + 1) * (cand * c + f);
              const double b = F * (cand * c + f) + ns * (y_max * c + f);
              const double sp = a > b ? a : b;
              if (sp < span) { span = sp; x_units = cand; }
            }
            if (x_units == 0) continue;
          }
          double cost = span + 0.5 * l2_clk;
          if (sl + ss > 1) cost += 8.0 * (sl + ss) * groups * static_cast<double>(r) * n / hbm_bytes_per_clk;
          if (cost < best) {
            best = cost;
            p.MB = mb;
            p.pair = pair != 0;
            p.s_long = sl;
            p.split_k = sl + ss;
            best_x = x_units;
          }
        }
      }
    }
  }
  const int cta_cols = p.MB * 128 * (p.pair ? 2 : 1);
  const int tiles_x = static_cast<int>((n + cta_cols - 1) / cta_cols);
  p.n_blocks = tiles_x * (p.pair ? 2 : 1);
  const int a_slabs = p.pair ? p.r_cta / 128 : p.r_cta / 64;
  p.bk = tc_bk(p.MB, a_slabs);
  p.k_blocks = static_cast<int>((T + p.bk - 1) / p.bk);
  p.gather = choose_gather(has_idx, opts, p.r_cta, tiles_x, m, r);
  p.kb_unit = p.gather == kOptCoop ? kCoopChunk / p.bk : 1;
  {
    // slice table: long slices of best_x units (or an equal cut), then the short ones
    const int U = (p.k_blocks + p.kb_unit - 1) / p.kb_unit;
    if (p.split_k > U) { p.split_k = U; if (p.s_long > U) p.s_long = U; }
    const int ss = p.split_k - p.s_long;
    int at = 0;
    for (int z = 0; z < p.split_k; ++z) {
      p.unit_begin[z] = at;
      if (ss == 0) at += U / p.split_k + (z < U % p.split_k ? 1 : 0);
      else if (z < p.s_long) at += best_x;
      else {
        const int y_total = U - p.s_long * best_x, zs = z - p.s_long;
        at += y_total / ss + (zs < y_total % ss ? 1 : 0);
      }
    }
    p.unit_begin[p.split_k] = U;
    for (int z = p.split_k + 1; z <= kTcMaxSlices; ++z) p.unit_begin[z] = U;
  }
  p.ctrl_bytes = p.gather == kOptCoop
                     ? round_up((kCoopCtrlInts + static_cast<size_t>(groups) *
                                                     ((T + kCoopChunk - 1) / kCoopChunk)) * sizeof(int), 256)
                     : 0;
  p.stages = tc_stages(p.MB, a_slabs);
  p.smem_bytes = static_cast<size_t>(p.stages) * tc_stage_bytes(p.MB, a_slabs) + 1024;
  p.ld_part = static_cast<long long>(round_up(static_cast<size_t>(n), 4));
  p.ag_bytes = p.gather == kOptPrepass || p.gather == kOptCoop
                   ? round_up(static_cast<size_t>(T) * p.r_pad * sizeof(__nv_bfloat16), 256)
                   : 0;
  p.part_bytes = p.split_k > 1
                     ? round_up(static_cast<size_t>(p.split_k) * r * p.ld_part * sizeof(float), 256)
                     : 0;
  return p;
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

// bf16 matrix [rows][cols] with row pitch ld (elements): box = {64 cols, bk rows}, 128B swizzle.
// Encoded on every call: a host-side cache keyed by (pointer, shape, pitch) was measured and
// saved nothing (40.8 us against 41.9 us of host time per batched call of four 60M layers).
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int bk) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  cuuint32_t box[2] = {64, static_cast<cuuint32_t>(bk)};
  cuuint32_t estr[2] = {1, 1};
  CUresult res = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (res != CUDA_SUCCESS) {
    fprintf(stderr, "grass: cuTensorMapEncodeTiled failed with %d\n", static_cast<int>(res));
    return false;
  }
  return true;
}

template <int MB, int NSLAB, bool PAIR, int GATHER>
int launch_tc_one(dim3 tile_grid, size_t smem, cudaStream_t s, const TcMaps& maps, TcParams p,
                  int kernel_id) {
  constexpr bool FUSED = GATHER != kGatherNone;   // the variants with eight extra warps
  static bool attr_set[64] = {false};
  static int max_workers[64] = {0};
  int dev = 0;
  GRASS_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return GRASS_ERR_INVALID_ARG;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(FUSED ? kTcThreads + kTcGatherThreads : kTcThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = PAIR ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (!attr_set[dev]) {
    GRASS_CUDA_TRY(cudaFuncSetAttribute(project_tc_kernel<MB, NSLAB, PAIR, GATHER>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kTcSmemBudget));
    // how many workers (CTAs, or CTA pairs) the device holds at once: one per SM / SM pair
    int workers = 0;
    if (PAIR) {
      cfg.gridDim = dim3(2 * kSmCount);
      GRASS_CUDA_TRY(cudaOccupancyMaxActiveClusters(&workers, project_tc_kernel<MB, NSLAB, PAIR, GATHER>,
                                                    &cfg));
    } else {
      GRASS_CUDA_TRY(cudaDeviceGetAttribute(&workers, cudaDevAttrMultiProcessorCount, dev));
    }
    if (workers < 1) workers = 1;
    max_workers[dev] = workers;
    attr_set[dev] = true;
  }
  // persistent launch: never more workers than are resident at once, each loops over its tiles
  p.tiles_x = static_cast<int>(tile_grid.x);
  p.tiles_y = static_cast<int>(tile_grid.y);
  const long long n_tiles = static_cast<long long>(tile_grid.x) * tile_grid.y * tile_grid.z;
  // (cooperative gather: every SM takes part in the gather, also those without a tile)
  const int workers = n_tiles < max_workers[dev] && GATHER != kGatherCoop && p.s_long == p.split_k
                          ? static_cast<int>(n_tiles) : max_workers[dev];
  cfg.gridDim = dim3(static_cast<unsigned>(PAIR ? 2 * workers : workers));
  {
    ProfileScope prof(kernel_id, s);
    GRASS_CUDA_TRY(cudaLaunchKernelEx(&cfg, project_tc_kernel<MB, NSLAB, PAIR, GATHER>, maps, p));
  }
  return GRASS_OK;
}

// (MB, NSLAB) with MB * 64 * NSLAB <= 512 TMEM columns; pairs need an even NSLAB.
// gather: kGatherNone / kGatherCta (tiles of at most 128 rows) / kGatherCoop.
int launch_tc(int MB, int nslab, bool pair, int gather, dim3 grid, size_t smem, cudaStream_t s,
              const TcMaps& maps, const TcParams& p, int kernel_id) {
#define GRASS_TC_CASE(mb, ns, pr, ga)                                                          \
  if (MB == mb && nslab == ns && pair == pr && gather == ga)                                   \
    return launch_tc_one<mb, ns, pr, ga>(grid, smem, s, maps, p, kernel_id)
#define GRASS_TC_BOTH(mb, ns, pr)                                                              \
  GRASS_TC_CASE(mb, ns, pr, kGatherNone);                                                      \
  GRASS_TC_CASE(mb, ns, pr, kGatherCoop)
  GRASS_TC_BOTH(1, 1, false); GRASS_TC_BOTH(1, 2, false); GRASS_TC_BOTH(1, 3, false);
  GRASS_TC_BOTH(1, 4, false); GRASS_TC_BOTH(1, 5, false); GRASS_TC_BOTH(1, 6, false);
  GRASS_TC_BOTH(1, 7, false); GRASS_TC_BOTH(1, 8, false);
  GRASS_TC_BOTH(2, 1, false); GRASS_TC_BOTH(2, 2, false); GRASS_TC_BOTH(2, 3, false);
  GRASS_TC_BOTH(2, 4, false);
  GRASS_TC_BOTH(4, 1, false); GRASS_TC_BOTH(4, 2, false);
  GRASS_TC_BOTH(1, 2, true); GRASS_TC_BOTH(1, 4, true); GRASS_TC_BOTH(1, 6, true);
  GRASS_TC_BOTH(1, 8, true);
  GRASS_TC_BOTH(2, 2, true); GRASS_TC_BOTH(2, 4, true); GRASS_TC_BOTH(4, 2, true);
  // in-CTA gather: at most 128 selected rows per tile
  GRASS_TC_CASE(1, 1, false, kGatherCta); GRASS_TC_CASE(2, 1, false, kGatherCta);
  GRASS_TC_CASE(4, 1, false, kGatherCta); GRASS_TC_CASE(1, 2, false, kGatherCta);
  GRASS_TC_CASE(2, 2, false, kGatherCta); GRASS_TC_CASE(4, 2, false, kGatherCta);
  GRASS_TC_CASE(1, 2, true, kGatherCta); GRASS_TC_CASE(2, 2, true, kGatherCta);
  GRASS_TC_CASE(4, 2, true, kGatherCta);
#undef GRASS_TC_BOTH
#undef GRASS_TC_CASE
  return GRASS_ERR_UNSUPPORTED;
}

size_t norm_part_bytes(int64_t m, int64_t n) {
  return round_up(static_cast<size_t>((n + 31) / 32) * round_up(static_cast<size_t>(m), 32) *
                      sizeof(float), 256);
}

// fp32 path: split the tokens when the output has too few 64 x 64 tiles to occupy the GPU.
struct Fp32Plan {
  int split;
  int64_t tokens_per_split;
  long long ld_part;
  size_t part_bytes;
};
Fp32Plan make_fp32_plan(int64_t T, int64_t n, int r) {
  Fp32Plan p;
  const int64_t tiles = ((n + kSimtBC - 1) / kSimtBC) * ((r + kSimtBJ - 1) / kSimtBJ);
  int64_t split = (2 * kSmCount + tiles - 1) / tiles;
  const int64_t max_split = (T + 2 * kSimtBT - 1) / (2 * kSimtBT);   // at least 32 tokens a slice
  if (split > max_split) split = max_split;
  if (split > 64) split = 64;
  if (split < 1) split = 1;
  int64_t per = (T + split - 1) / split;
  per = (per + kSimtBT - 1) / kSimtBT * kSimtBT;
  p.tokens_per_split = per;
  p.split = static_cast<int>((T + per - 1) / per);
  p.ld_part = static_cast<long long>(round_up(static_cast<size_t>(n), 4));
  p.part_bytes = p.split > 1
                     ? round_up(static_cast<size_t>(p.split) * r * p.ld_part * sizeof(float), 256)
                     : 0;
  return p;
}

// Row-norm mode.  The squares must be taken of complete dot products, so the fused epilogue
// needs an unsplit token sum; that is the plan whenever the dense m x n output has enough tiles
// to occupy the GPU (every LLaMA shape from 1B up).  A small gradient (few tiles) would leave
// most SMs idle, so it is computed with the usual token split into fp32 partials -- small by
// the same token -- and splitk_rownorms_kernel sums, squares and reduces them.
TcPlan make_norms_plan(int64_t T, int64_t m, int64_t n) {
  const PlanOpts none;
  const TcPlan fused = make_plan(T, m, n, static_cast<int>(m), false, none, true);
  if (static_cast<int64_t>(fused.n_blocks) * fused.r_blocks >= 120) return fused;
  return make_plan(T, m, n, static_cast<int>(m), false, none, false);
}

// Bytes of workspace a plan needs for `count` layers: [control block][per layer: gathered operand,
// split-K partials].
size_t plan_ws_bytes(const TcPlan& plan, int count) {
  return plan.ctrl_bytes + (plan.ag_bytes + plan.part_bytes) * static_cast<size_t>(count);
}

// Projection of `count` same-shaped layers in one set of launches (count = 1 for the plain
// call).  norms != NULL (count must be 1): row-norm mode (idx NULL, r == m): the GEMM's epilogue
// reduces squares instead of storing the gradient, then the partial sums are finalised.
int project_bf16(int count, const void* const* dY, int64_t lddy, const void* const* X, int64_t ldx,
                 int64_t T, int64_t m, int64_t n, const int32_t* const* idx,
                 const float* const* rho, int r, float* const* Gc, int64_t ldgc, float* norms,
                 void* ws, size_t ws_bytes, const PlanOpts& opts, cudaStream_t s) {
  if (count < 1 || count > kTcMaxGroup || (norms != nullptr && count != 1))
    return GRASS_ERR_INVALID_ARG;
  const bool gather = idx != nullptr && idx[0] != nullptr;
  for (int g = 0; g < count; ++g) {
    if (dY[g] == nullptr || X[g] == nullptr || (norms == nullptr && Gc[g] == nullptr))
      return GRASS_ERR_INVALID_ARG;
    if (gather != (idx != nullptr && idx[g] != nullptr)) return GRASS_ERR_INVALID_ARG;
    if (!aligned_to(X[g], 16) || ldx % 8 != 0) return GRASS_ERR_ALIGNMENT;
    if (!gather && (!aligned_to(dY[g], 16) || lddy % 8 != 0)) return GRASS_ERR_ALIGNMENT;
  }
  const TcPlan plan = norms != nullptr ? make_norms_plan(T, m, n)
                                       : make_plan(T, m, n, r, gather, opts, false, count);
  if (plan.gather == kOptPrepass && T > 65535LL * kGatherTokens)
    return GRASS_ERR_UNSUPPORTED;                                            // pre-pass grid.y
  if (plan.unit_begin[plan.split_k] > 65535) return GRASS_ERR_UNSUPPORTED;   // 16-bit slice table
  const bool fused_norms = norms != nullptr && plan.split_k == 1;
  const size_t per_layer = fused_norms ? norm_part_bytes(m, n) : plan.ag_bytes + plan.part_bytes;
  const size_t need = plan.ctrl_bytes + per_layer * count;
  if (need > 0 && (ws == nullptr || !aligned_to(ws, 256) || ws_bytes < need))
    return GRASS_ERR_WORKSPACE;
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);

  TcMaps maps;
  GatherGroup gg;
  float* part[kTcMaxGroup];
  char* const layers_ws = static_cast<char*>(ws) + plan.ctrl_bytes;
  for (int g = 0; g < count; ++g) {
    char* wsp = layers_ws + per_layer * g;
    if (!make_map(&maps.x[g], X[g], T, n, ldx, plan.bk)) return GRASS_ERR_CUDA;
    gg.dY[g] = static_cast<const __nv_bfloat16*>(dY[g]);
    gg.idx[g] = gather ? idx[g] : nullptr;
    gg.Ag[g] = nullptr;
    if (plan.gather == kOptCta) {
      maps.a[g] = maps.x[g];          // unused by the kernel
    } else if (plan.gather == kOptPrepass || plan.gather == kOptCoop) {
      gg.Ag[g] = reinterpret_cast<__nv_bfloat16*>(wsp);
      if (!make_map(&maps.a[g], gg.Ag[g], T, plan.r_pad, plan.r_pad, plan.bk)) return GRASS_ERR_CUDA;
      wsp += plan.ag_bytes;
    } else {
      if (!make_map(&maps.a[g], dY[g], T, m, lddy, plan.bk)) return GRASS_ERR_CUDA;
    }
    part[g] = reinterpret_cast<float*>(wsp);
  }
  for (int g = count; g < kTcMaxGroup; ++g) {
    maps.x[g] = maps.x[0];
    maps.a[g] = maps.a[0];
    gg.dY[g] = nullptr; gg.idx[g] = nullptr; gg.Ag[g] = nullptr;
  }
  if (plan.gather == kOptPrepass) {
    ProfileScope prof(GRASS_K_GATHER, s);
    const int ni = plan.r_pad >= 256 ? 8 : plan.r_pad / 32;   // r_pad is a multiple of 64
    dim3 ggrid(static_cast<unsigned>((plan.r_pad + 32 * ni - 1) / (32 * ni)),
               static_cast<unsigned>((T + kGatherTokens - 1) / kGatherTokens),
               static_cast<unsigned>(count));
    gather_cols_kernel<<<ggrid, kGatherThreads, 0, s>>>(gg, lddy, static_cast<int>(T),
                                                        static_cast<int>(m), r, plan.r_pad, ni,
                                                        status);
    GRASS_LAUNCH_CHECK();
  }

  TcParams p;
  p.T = static_cast<int>(T);
  p.n = static_cast<int>(n);
  p.r = r;
  p.k_blocks = plan.k_blocks;
  p.split_k = plan.split_k;
  p.s_long = plan.s_long;
  p.kb_unit = plan.kb_unit;
  p.groups = count;
  for (int z = 0; z <= kTcMaxSlices; ++z) p.unit_begin[z] = static_cast<unsigned short>(plan.unit_begin[z]);
  p.status = status;
  p.norm_part = fused_norms ? part[0] : nullptr;
  const bool in_kernel = plan.gather == kOptCta || plan.gather == kOptCoop;
  for (int g = 0; g < kTcMaxGroup; ++g) {
    const int gi = g < count ? g : 0;
    p.dY[g] = in_kernel ? gg.dY[gi] : nullptr;
    p.idx[g] = in_kernel ? gg.idx[gi] : nullptr;
    p.Ag[g] = plan.gather == kOptCoop ? gg.Ag[gi] : nullptr;
  }
  p.lddy = lddy;
  p.m = static_cast<int>(m);
  p.r_pad = plan.r_pad;
  p.coop_ctrl = nullptr;
  p.coop_warps = opts.gather_warps > 0 ? opts.gather_warps : 8;
  p.coop_chunks = static_cast<int>((T + kCoopChunk - 1) / kCoopChunk);
  p.coop_cg = (plan.r_pad + kCoopCols - 1) / kCoopCols;
  p.coop_pmax_long = p.coop_pmax_short = 0;
  for (int z = 0; z < plan.split_k; ++z) {
    const int units = plan.unit_begin[z + 1] - plan.unit_begin[z];
    int& pm = z < plan.s_long ? p.coop_pmax_long : p.coop_pmax_short;
    if (units > pm) pm = units;
  }
  if (plan.gather == kOptCoop) {
    // queue head and per-chunk counters start at zero for every launch
    p.coop_ctrl = static_cast<int*>(ws);
    GRASS_CUDA_TRY(cudaMemsetAsync(ws, 0, plan.ctrl_bytes, s));
  }
  p.ld_norm = static_cast<long long>(round_up(static_cast<size_t>(m), 32));
  for (int g = 0; g < kTcMaxGroup; ++g) {
    const int gi = g < count ? g : 0;
    if (plan.split_k == 1) {
      p.out[g] = Gc != nullptr ? Gc[gi] : nullptr;   // unused in row-norm mode
      p.rho[g] = rho != nullptr ? rho[gi] : nullptr;
    } else {
      p.out[g] = part[gi];
      p.rho[g] = nullptr;
    }
  }
  p.ld_out = plan.split_k == 1 ? ldgc : plan.ld_part;
  p.split_stride = plan.split_k == 1 ? 0 : static_cast<long long>(r) * plan.ld_part;
  // tile space handed to the persistent kernel (x counts pairs of CTAs in pair mode)
  dim3 grid(static_cast<unsigned>(plan.pair ? plan.n_blocks / 2 : plan.n_blocks),
            static_cast<unsigned>(plan.r_blocks), static_cast<unsigned>(plan.split_k * count));

  const int kernel_gather = plan.gather == kOptCta ? kGatherCta
                            : plan.gather == kOptCoop ? kGatherCoop : kGatherNone;
  const int rc = launch_tc(plan.MB, plan.r_cta / 64, plan.pair, kernel_gather, grid, plan.smem_bytes,
                           s, maps, p, gather ? GRASS_K_PROJECT_TC : GRASS_K_PROJECT_TC_DENSE);
  if (rc != GRASS_OK) return rc;
  if (norms != nullptr) {
    ProfileScope prof(GRASS_K_ROW_NORMS, s);
    if (fused_norms)
      norms_finalize_kernel<<<static_cast<unsigned>((m + 255) / 256), 256, 0, s>>>(
          p.norm_part, p.ld_norm, static_cast<int>((n + 31) / 32), static_cast<int>(m), norms);
    else
      splitk_rownorms_kernel<<<static_cast<unsigned>(m), 256, 0, s>>>(
          part[0], plan.ld_part, p.split_stride, plan.split_k, static_cast<int>(m),
          static_cast<int>(n), norms);
    GRASS_LAUNCH_CHECK();
    return GRASS_OK;
  }
  if (plan.split_k > 1) {
    ReduceGroup rg;
    int vec = (n % 4 == 0) && (ldgc % 4 == 0);
    for (int g = 0; g < kTcMaxGroup; ++g) {
      const int gi = g < count ? g : 0;
      rg.part[g] = part[gi];
      rg.rho[g] = rho != nullptr ? rho[gi] : nullptr;
      rg.Gc[g] = Gc[gi];
      vec = vec && aligned_to(Gc[gi], 16);
    }
    const long long work = static_cast<long long>(r) * (vec ? n / 4 : n);
    long long blocks = (work + 255) / 256;
    if (blocks > kSmCount * 32) blocks = kSmCount * 32;
    ProfileScope prof(GRASS_K_SPLITK_REDUCE, s);
    splitk_reduce_kernel<<<dim3(static_cast<unsigned>(blocks), static_cast<unsigned>(count)), 256, 0,
                           s>>>(rg, plan.ld_part, p.split_stride, plan.split_k, r,
                                static_cast<int>(n), ldgc, vec);
    GRASS_LAUNCH_CHECK();
  }
  return GRASS_OK;
}

void describe_plan(const TcPlan& plan, int count, grass_project_plan_t* out) {
  out->gather = plan.gather;
  out->rows_per_tile = plan.r_cta;
  out->row_blocks = plan.r_blocks;
  out->n_blocks_per_cta = plan.MB;
  out->ctas_per_slice = plan.n_blocks * plan.r_blocks * count;
  out->cta_pair = plan.pair ? 1 : 0;
  out->token_slices = plan.split_k;
  out->short_slices = plan.split_k - plan.s_long;
  out->long_slice_tokens = (plan.unit_begin[1] - plan.unit_begin[0]) * plan.kb_unit * plan.bk;
  out->tokens_per_stage = plan.bk;
  out->stages = plan.stages;
  out->workspace_bytes = plan_ws_bytes(plan, count) + 256;
}

}  // namespace
}  // namespace grass

extern "C" size_t grass_project_workspace_bytes(int64_t T, int64_t m, int64_t n, int32_t r,
                                                int dt) {
  if (T < 1 || m < 1 || n < 1 || r < 1) return 0;
  if (dt != GRASS_BF16) return grass::make_fp32_plan(T, n, r).part_bytes + 256;
  // covers the call with and without idx (the dense form needs no gathered operand)
  const size_t with_idx = grass::plan_ws_bytes(grass::make_plan(T, m, n, r, true, grass::PlanOpts()), 1);
  const size_t dense = grass::plan_ws_bytes(grass::make_plan(T, m, n, r, false, grass::PlanOpts()), 1);
  return (with_idx > dense ? with_idx : dense) + 256;
}

namespace grass {
namespace {
int project_fp32(const void* dY, int64_t lddy, const void* X, int64_t ldx, int64_t T, int64_t m,
                 int64_t n, const int32_t* idx, const float* rho, int32_t r, float* Gc,
                 int64_t ldgc, void* ws, size_t ws_bytes, cudaStream_t s) {
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  const Fp32Plan fp = make_fp32_plan(T, n, r);
  if (fp.split > 1 && (ws == nullptr || !aligned_to(ws, 256) || ws_bytes < fp.part_bytes))
    return GRASS_ERR_WORKSPACE;
  dim3 grid(static_cast<unsigned>((n + kSimtBC - 1) / kSimtBC),
            static_cast<unsigned>((r + kSimtBJ - 1) / kSimtBJ), static_cast<unsigned>(fp.split));
  float* out = fp.split > 1 ? static_cast<float*>(ws) : Gc;
  const int64_t ld_out = fp.split > 1 ? fp.ld_part : ldgc;
  {
    ProfileScope prof(GRASS_K_PROJECT_FP32, s);
    project_simt_kernel<float><<<grid, kSimtThreads, 0, s>>>(
        static_cast<const float*>(dY), lddy, static_cast<const float*>(X), ldx, T, m, n, idx, rho, r,
        out, ld_out, fp.tokens_per_split, static_cast<int64_t>(r) * fp.ld_part, status);
  }
  GRASS_LAUNCH_CHECK();
  if (fp.split > 1) {
    const int vec = (n % 4 == 0) && (ldgc % 4 == 0) && aligned_to(Gc, 16);
    const long long work = static_cast<long long>(r) * (vec ? n / 4 : n);
    long long blocks = (work + 255) / 256;
    if (blocks > kSmCount * 32) blocks = kSmCount * 32;
    ProfileScope prof(GRASS_K_SPLITK_REDUCE, s);
    ReduceGroup rg;
    for (int g = 0; g < kTcMaxGroup; ++g) { rg.part[g] = out; rg.rho[g] = rho; rg.Gc[g] = Gc; }
    splitk_reduce_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(
        rg, fp.ld_part, static_cast<long long>(r) * fp.ld_part, fp.split, r, static_cast<int>(n),
        ldgc, vec);
    GRASS_LAUNCH_CHECK();
  }
  return GRASS_OK;
}
}  // namespace
}  // namespace grass

extern "C" int grass_project_grad(const void* dY, int64_t lddy, const void* X, int64_t ldx, int dt,
                                  int64_t T, int64_t m, int64_t n, const int32_t* idx,
                                  const float* rho, int32_t r, float* Gc, int64_t ldgc, void* ws,
                                  size_t ws_bytes, void* stream) {
  using namespace grass;
  if (dY == nullptr || X == nullptr || Gc == nullptr || T < 1 || m < 1 || n < 1 || r < 1 ||
      lddy < m || ldx < n || ldgc < n || T > 0x7fffffffLL || m > 0x7fffffffLL ||
      n > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  if (idx == nullptr && r != m) return GRASS_ERR_INVALID_ARG;
  if (r > m) return GRASS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == GRASS_BF16)
    return project_bf16(1, &dY, lddy, &X, ldx, T, m, n, idx != nullptr ? &idx : nullptr, &rho, r,
                        &Gc, ldgc, nullptr, ws, ws_bytes, PlanOpts(), s);
  if (dt != GRASS_F32) return GRASS_ERR_UNSUPPORTED;
  return project_fp32(dY, lddy, X, ldx, T, m, n, idx, rho, r, Gc, ldgc, ws, ws_bytes, s);
}

extern "C" size_t grass_project_batched_workspace_bytes(int32_t count, int64_t T, int64_t m,
                                                        int64_t n, int32_t r) {
  if (count < 1 || count > grass::kTcMaxGroup || T < 1 || m < 1 || n < 1 || r < 1) return 0;
  const grass::TcPlan plan = grass::make_plan(T, m, n, r, true, grass::PlanOpts(), false, count);
  return grass::plan_ws_bytes(plan, count) + 256;
}

extern "C" int grass_project_grad_batched(int32_t count, const void* const* dY, int64_t lddy,
                                          const void* const* X, int64_t ldx, int64_t T, int64_t m,
                                          int64_t n, const int32_t* const* idx,
                                          const float* const* rho, int32_t r, float* const* Gc,
                                          int64_t ldgc, void* ws, size_t ws_bytes, void* stream) {
  return grass_project_grad_ex(count, dY, lddy, X, ldx, T, m, n, idx, rho, r, Gc, ldgc, ws, ws_bytes,
                               nullptr, stream);
}

extern "C" int grass_project_plan(int32_t count, int64_t T, int64_t m, int64_t n, int32_t r,
                                  const grass_project_opts_t* opts, grass_project_plan_t* plan) {
  using namespace grass;
  if (plan == nullptr || count < 1 || count > kTcMaxGroup || T < 1 || m < 1 || n < 1 || r < 1 ||
      r > m || T > 0x7fffffffLL || m > 0x7fffffffLL || n > 0x7fffffffLL || !opts_ok(opts))
    return GRASS_ERR_INVALID_ARG;
  describe_plan(make_plan(T, m, n, r, true, to_plan_opts(opts), false, count), count, plan);
  return GRASS_OK;
}

extern "C" int grass_project_grad_ex(int32_t count, const void* const* dY, int64_t lddy,
                                     const void* const* X, int64_t ldx, int64_t T, int64_t m,
                                     int64_t n, const int32_t* const* idx, const float* const* rho,
                                     int32_t r, float* const* Gc, int64_t ldgc, void* ws,
                                     size_t ws_bytes, const grass_project_opts_t* opts,
                                     void* stream) {
  using namespace grass;
  if (count < 1 || count > kTcMaxGroup || dY == nullptr || X == nullptr || idx == nullptr ||
      Gc == nullptr || T < 1 || m < 1 || n < 1 || r < 1 || r > m || lddy < m || ldx < n ||
      ldgc < n || T > 0x7fffffffLL || m > 0x7fffffffLL || n > 0x7fffffffLL || !opts_ok(opts))
    return GRASS_ERR_INVALID_ARG;
  for (int g = 0; g < count; ++g)
    if (idx[g] == nullptr) return GRASS_ERR_INVALID_ARG;
  return project_bf16(count, dY, lddy, X, ldx, T, m, n, idx, rho, r, Gc, ldgc, nullptr, ws, ws_bytes,
                      to_plan_opts(opts), static_cast<cudaStream_t>(stream));
}

extern "C" size_t grass_grad_row_norms_workspace_bytes(int64_t T, int64_t m, int64_t n, int dt) {
  if (m < 1 || n < 1 || T < 1) return 0;
  if (dt == GRASS_BF16) {
    const grass::TcPlan plan = grass::make_norms_plan(T, m, n);
    return (plan.split_k == 1 ? grass::norm_part_bytes(m, n) : plan.part_bytes) + 256;
  }
  return grass::round_up(static_cast<size_t>(m) * n * sizeof(float), 256) +
         grass::make_fp32_plan(T, n, static_cast<int>(m)).part_bytes + 256;
}

extern "C" int grass_grad_row_norms(const void* dY, int64_t lddy, const void* X, int64_t ldx, int dt,
                                    int64_t T, int64_t m, int64_t n, float* norms, void* ws,
                                    size_t ws_bytes, void* stream) {
  using namespace grass;
  if (dY == nullptr || X == nullptr || norms == nullptr || T < 1 || m < 1 || n < 1 || lddy < m ||
      ldx < n || T > 0x7fffffffLL || m > 0x7fffffffLL || n > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == GRASS_BF16)
    return project_bf16(1, &dY, lddy, &X, ldx, T, m, n, nullptr, nullptr, static_cast<int>(m),
                        nullptr, 0, norms, ws, ws_bytes, PlanOpts(), s);
  if (dt != GRASS_F32) return GRASS_ERR_UNSUPPORTED;
  // fp32 path: the (small) gradient is formed in the workspace and reduced by grass_row_norms
  if (ws == nullptr || !aligned_to(ws, 256) ||
      ws_bytes < grass_grad_row_norms_workspace_bytes(T, m, n, dt) - 256)
    return GRASS_ERR_WORKSPACE;
  float* G = static_cast<float*>(ws);
  const size_t g_bytes = round_up(static_cast<size_t>(m) * n * sizeof(float), 256);
  const int rc = grass_project_grad(dY, lddy, X, ldx, dt, T, m, n, nullptr, nullptr,
                                    static_cast<int32_t>(m), G, n, static_cast<char*>(ws) + g_bytes,
                                    ws_bytes - g_bytes, stream);
  if (rc != GRASS_OK) return rc;
  return grass_row_norms(G, GRASS_F32, m, n, n, norms, stream);
}
