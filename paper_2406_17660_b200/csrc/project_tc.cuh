// bf16 tensor-core path of grass_project_grad (Section 3.1 of the GRASS paper):
//   Gc[j, c] = rho_j * sum_t dY[t, idx_j] * X[t, c].
//
// The contraction runs over tokens (T = 32K..64K) while the output r x n is
// small, so the kernel is organised around one rule: read X once.  A CTA owns
// an output tile of (MB * 128) columns of n by r_cta = 64 * NSLAB selected rows
// with MB * r_cta <= 512, i.e. up to all 512 fp32 TMEM columns, and a slice of
// the tokens (split-K); every X element it loads meets all r_cta rows.
//
// Operand roles are swapped with respect to the formula so that neither input
// needs a transpose in HBM:  D^T[c, j] = sum_t X[t, c] * A[t, j]  with
//   A-operand = X tile      (M = 128 columns of n, MN-major: c contiguous)
//   B-operand = gathered dY (N = up to 256 selected rows, MN-major: j contiguous)
// Both are staged by TMA as slabs of [BK tokens][64 elements] (BK = 64 or 32)
// with the 128-byte swizzle, which is the canonical MN-major UMMA layout.  TMEM lane = c, TMEM
// column = j, so the epilogue's tcgen05.ld hands each warp 32 consecutive c for
// one j per register: every store instruction writes 128 contiguous bytes.
//
// The kernel is persistent: at most one CTA (pair) per SM (pair), each looping over tiles, so
// TMEM, barriers and the TMA ring are set up once and the producer keeps the ring full across
// tile boundaries; a "TMEM free" barrier returns the accumulators from the epilogue warps to
// the MMA issuer between tiles.
//
// GATHER selects how the selected dY columns reach the B operand:
//   kGatherNone  the operand is read by TMA from a matrix that already exists (dY itself for
//                the dense gradient, or the output of the stand-alone gather_cols_kernel);
//   kGatherCta   eight extra warps pick dY[t, idx_j] themselves and write the bytes into this
//                CTA's B-operand slabs (generic-proxy stores in the swizzled layout, proxy
//                fence, arrive on "full"): for small, densely picked tiles;
//   kGatherCoop  eight extra warps in EVERY CTA of the grid share the gather of the whole launch:
//                they take (token chunk, column group) items from one queue in the order the
//                GEMM consumes them, write the picked columns to the token-major operand matrix
//                in the workspace (it stays in L2) and publish a per-chunk counter; a CTA's TMA
//                producer waits for the counter of a chunk before it loads from it.  The gather
//                is done once per launch instead of once per n-tile, and it overlaps the MMAs
//                instead of preceding them.  Gather warps never wait on anything, so progress
//                does not depend on which CTAs are resident.
//
// Warp roles (320 threads): warp 0 = TMA producer (one lane per slab), warp 1 =
// TMEM owner + single-thread MMA issuer, warps 2..9 = epilogue (warp w reads
// TMEM lanes 32*(w%4)..+31; the two warps of a lane quarter alternate over the
// 32-column chunks).  A lone issuing thread retires roughly one dependent
// instruction every 4-5 clocks, so the per-stage instruction count of the
// producer and of the MMA issuer bounds the pipeline: tile shape and stage
// count are template parameters so that every descriptor is a constant plus
// the stage offset and the loops unroll.
//
// PAIR = true runs two CTAs of a cluster as one tcgen05 "CTA pair"
// (cta_group::2): M = 256 (each CTA holds its own 128 columns of n in its own
// TMEM), and the B operand is split between the two CTAs, each staging only
// half of the selected rows.  Shared-memory traffic per SM drops from
// 96 B/clk of MMA reads + 80 B/clk of TMA writes (above the 128 B/clk an SM
// can move) to 64 + 48.  The even CTA issues the MMAs for both; both CTAs' TMA
// loads report to the even CTA's "full" barrier; tcgen05.commit signals the
// "empty" and "accumulator ready" barriers of both CTAs.  No load is multicast.
// Every mbarrier wait is bounded; on expiry the CTA records GRASS_ERR_TIMEOUT,
// drains what it has in flight (bounded again), frees its TMEM and returns.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace grass {

// Tokens per pipeline stage: 64 where at least four such stages fit, else 32.  A stage costs
// the two issuing threads a fixed number of instructions (barrier wait, fence, commit, copy
// issue); with 64 tokens that cost is spread over twice as many MMAs (234 -> 193 us on the
// LLaMA-7B q shape).  A slab is [BK tokens][64 bf16].
constexpr int kTcThreads = 320;
constexpr int kTcGatherThreads = 256;   // extra warps of the in-kernel gather variant
constexpr int kTcMaxStages = 8;
constexpr int kTcSmemBudget = 227 * 1024 - 1024;  // dynamic part; the rest holds the barriers
constexpr long long kTcWaitLimit = 2000000000LL;  // SM clocks (~1 s)
constexpr long long kTcDrainLimit = 200000000LL;  // give-up path: wait for work in flight

__host__ __device__ constexpr int tc_stage_bytes_bk(int MB, int A_SLABS, int BK) {
  return (2 * MB + A_SLABS) * BK * 128;
}
__host__ __device__ constexpr int tc_bk(int MB, int A_SLABS) {
  return (kTcSmemBudget - 1024) / tc_stage_bytes_bk(MB, A_SLABS, 64) >= 4 ? 64 : 32;
}
__host__ __device__ constexpr int tc_stage_bytes(int MB, int A_SLABS) {
  return tc_stage_bytes_bk(MB, A_SLABS, tc_bk(MB, A_SLABS));
}
__host__ __device__ constexpr int tc_stages(int MB, int A_SLABS) {
  return (kTcSmemBudget - 1024) / tc_stage_bytes(MB, A_SLABS) > kTcMaxStages
             ? kTcMaxStages
             : (kTcSmemBudget - 1024) / tc_stage_bytes(MB, A_SLABS);
}

constexpr int kTcMaxGroup = 8;
constexpr int kTcMaxSlices = 64;    // token slices per layer

constexpr int kGatherNone = 0, kGatherCta = 1, kGatherCoop = 2;
// Cooperative gather: tokens per chunk (one readiness counter each), columns per item, and the
// parts (one warp each) a chunk's tokens are dealt into.  Token slices of the GEMM start on
// chunk borders in this mode.
constexpr int kCoopChunk = 128;
constexpr int kCoopCols = 256;
constexpr int kCoopParts = 16;
constexpr int kCoopCtrlInts = 64;     // control block: [0] queue head, flags from [kCoopCtrlInts]

// The X and gathered-dY tensor maps of every layer of the group (kernel parameter space).
struct TcMaps {
  CUtensorMap x[kTcMaxGroup];
  CUtensorMap a[kTcMaxGroup];
};

struct TcParams {
  int T, n, r;          // logical sizes
  int k_blocks;         // ceil(T / tokens per stage)
  int split_k;          // token slices per layer; slice z covers the units
                        // [unit_begin[z], unit_begin[z + 1]) of kb_unit token blocks each
  int s_long;           // the first s_long slices are "long", the others "short" (see the
                        // tile schedule in the kernel); s_long == split_k: all alike
  int kb_unit;
  unsigned short unit_begin[kTcMaxSlices + 1];
  int tiles_x, tiles_y; // output tiles of one layer: n-tiles (per pair if PAIR), row blocks
  int groups;           // up to kTcMaxGroup same-shaped layers share one launch
  float* out[kTcMaxGroup];        // split_k == 1: Gc, else partials [split][r][ld_out]
  long long ld_out;     // row pitch of out, elements
  long long split_stride;  // elements between partials of consecutive splits
  const float* rho[kTcMaxGroup];  // applied here only when split_k == 1 (entries may be NULL)
  // in-kernel gather variant: the selected columns are picked straight out of dY
  const __nv_bfloat16* dY[kTcMaxGroup];
  const int32_t* idx[kTcMaxGroup];
  long long lddy;
  int m;
  // cooperative gather: operand matrices [T][r_pad] being filled, control block, item space
  __nv_bfloat16* Ag[kTcMaxGroup];
  int r_pad;
  int* coop_ctrl;
  int coop_chunks;      // chunks per layer = ceil(T / kCoopChunk)
  int coop_cg;          // column groups = ceil(r_pad / kCoopCols)
  int coop_pmax_long, coop_pmax_short;   // most chunks in one long / short token slice
  int coop_warps;       // gather warps per CTA that take part (1..8)
  float* norm_part;     // non-NULL: row-norm mode.  Nothing of D is stored; instead
                        // norm_part[g * ld_norm + j] = sum of D[j, c]^2 over the 32 columns c of group g
  long long ld_norm;
  int* status;
};

// Sum 32 per-lane values across the warp, all 32 at once: on return lane l holds
// sum over lanes of x[l].  31 shuffles (halving exchange) instead of 32 x 5.
__device__ __forceinline__ float warp_transpose_sum(float (&x)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < off; ++k) {
      const float send = upper ? x[k] : x[k + off];
      const float keep = upper ? x[k + off] : x[k];
      x[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return x[0];
}

// dY[t, rows[i]] for 32 (token, column) pairs per lane in flight, written to the operand matrix.
// Lane l carries columns col0 + 32 i + l, i < NI; tokens tok0, tok0 + kCoopParts, ...
template <int NI>
__device__ __forceinline__ void coop_gather_part(const unsigned short* __restrict__ src,
                                                 long long lddy, unsigned short* __restrict__ dst,
                                                 int r_pad, int col0, const int (&rows)[8], int tok0,
                                                 int T, int lane, int* publish) {
  constexpr int TU = (32 / NI) < (kCoopChunk / kCoopParts) ? (32 / NI) : (kCoopChunk / kCoopParts);   // tokens per batch of loads
  constexpr int NTOK = kCoopChunk / kCoopParts;           // tokens of this part
  // Every load is unconditional (rows and tokens clamped to valid ones, the value discarded at
  // the store): a load under a per-lane condition would be followed by a select on its result,
  // and the warp would wait for each load before issuing the next.
  int safe[NI];
#pragma unroll
  for (int i = 0; i < NI; ++i) safe[i] = rows[i] >= 0 ? rows[i] : 0;
#pragma unroll 1
  for (int k0 = 0; k0 < NTOK; k0 += TU) {
    unsigned short v[TU][NI];
#pragma unroll
    for (int u = 0; u < TU; ++u) {
      const int tok = tok0 + (k0 + u) * kCoopParts;
      const unsigned short* line = src + static_cast<long long>(tok < T ? tok : T - 1) * lddy;
#pragma unroll
      for (int i = 0; i < NI; ++i) v[u][i] = ptx::ld_nc_na_u16(line + safe[i]);
    }
    if (publish != nullptr) {
      // the previous item's stores (all lanes, program order + warp barrier) become visible
      // before its counter moves; the fence's wait hides behind the loads just issued
      __syncwarp();
      if (lane == 0) ptx::flag_arrive_release(publish);
      publish = nullptr;
    }
#pragma unroll
    for (int u = 0; u < TU; ++u) {
      const int tok = tok0 + (k0 + u) * kCoopParts;
      unsigned short* out = dst + static_cast<long long>(tok) * r_pad + col0 + lane;
#pragma unroll
      for (int i = 0; i < NI; ++i)
        if (tok < T && col0 + 32 * i + lane < r_pad) out[32 * i] = rows[i] >= 0 ? v[u][i] : 0;
    }
  }
}

template <int MB, int NSLAB, bool PAIR, int GATHER>
__global__ void __launch_bounds__(GATHER != kGatherNone ? kTcThreads + kTcGatherThreads : kTcThreads, 1)
project_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
  constexpr bool FUSED = GATHER == kGatherCta;
  constexpr bool COOP = GATHER == kGatherCoop;
  constexpr int R_CTA = 64 * NSLAB;          // selected rows per CTA tile (per pair if PAIR)
  constexpr int X_SLABS = 2 * MB;
  constexpr int A_SLABS = PAIR ? NSLAB / 2 : NSLAB;   // slabs of the gathered operand this CTA stages
  constexpr int N_SLABS = X_SLABS + A_SLABS;
  constexpr int kTcBK = tc_bk(MB, A_SLABS);           // tokens per stage
  constexpr int kTcSlabBytes = kTcBK * 128;
  constexpr int STAGE_BYTES = tc_stage_bytes(MB, A_SLABS);
  // FUSED: the gathered operand is not copied by TMA but picked out of dY by the gather warps,
  // so only the X slabs are TMA traffic; every gather warp of the pair reports to "full"
  constexpr int TMA_SLABS = FUSED ? X_SLABS : N_SLABS;
  constexpr int TMA_BYTES = TMA_SLABS * kTcSlabBytes;
  constexpr int FULL_ARRIVALS = 1 + (FUSED ? (kTcGatherThreads / 32) * (PAIR ? 2 : 1) : 0);
  constexpr int STAGES = tc_stages(MB, A_SLABS);
  constexpr int UMMA_M = PAIR ? 256 : 128;
  constexpr int C_STEP = PAIR ? 256 : 128;   // columns between this CTA's consecutive blocks
  static_assert(MB * R_CTA <= 512, "accumulators exceed TMEM");
  static_assert(N_SLABS <= 32, "one producer lane per slab");
  static_assert(!PAIR || NSLAB % 2 == 0, "a CTA pair splits the selected rows in halves of 64k");

  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kTcMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kTcMaxStages];
  __shared__ __align__(8) uint64_t bar_accum;       // accumulators of the current tile complete
  __shared__ __align__(8) uint64_t bar_tmem_free;   // every epilogue warp has read them out
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  const int rank = PAIR ? static_cast<int>(ptx::cluster_ctarank()) : 0;
  // Persistent workers and the tile schedule.  A tile is (n-tile bx, row block by, layer, token
  // slice z); a worker is a CTA, or a CTA pair.  With W workers and N tiles of equal length the
  // last wave is only partly filled whenever W does not divide N.  The host therefore cuts
  // the tokens into s_long long slices and (optionally) a few short ones: the long tiles are
  // dealt round-robin (worker w takes w, w + W, ...: the order a plain grid would be dispatched
  // in, so concurrent workers sweep the tokens together and share operands through L2), and the
  // R = N_long mod W workers that got one long tile more than the others are done; the other
  // W - R workers share the short tiles round-robin.  The slice lengths are chosen so that both
  // kinds of worker finish together.  Every tile writes its own split-K partial, so the
  // result does not depend on which worker ran it.
  const int n_workers = PAIR ? static_cast<int>(gridDim.x >> 1) : static_cast<int>(gridDim.x);
  const int worker = PAIR ? static_cast<int>(blockIdx.x >> 1) : static_cast<int>(blockIdx.x);
  const int txy = p.tiles_x * p.tiles_y;
  const int s_short = p.split_k - p.s_long;
  const int n_long = txy * p.groups * p.s_long, n_short = txy * p.groups * s_short;
  const int sched_R = n_long % n_workers;
  const int short_workers = sched_R > 0 ? n_workers - sched_R : n_workers;
  const int my_long = worker < n_long ? (n_long - worker + n_workers - 1) / n_workers : 0;

  // the k-th tile of this worker (identical in every role); false when there is none
  struct Tile { int c_base, r0, grp, z, kb_begin, kb_count; };
  auto sched = [&](int k, Tile& t) -> bool {
    int L, sl, z0;
    if (k < my_long) {
      L = worker + k * n_workers;
      sl = p.s_long;
      z0 = 0;
    } else {
      if (sched_R > 0 && worker < sched_R) return false;
      L = (sched_R > 0 ? worker - sched_R : worker) + (k - my_long) * short_workers;
      if (L >= n_short) return false;
      sl = s_short;
      z0 = p.s_long;
    }
    const int bx = L % p.tiles_x;
    const int rest = L / p.tiles_x;
    const int by = rest % p.tiles_y, bz = rest / p.tiles_y;
    // PAIR: CTA `rank` of the pair owns, for each of its MB blocks, the 128 columns
    // pair_base + (mb * 2 + rank) * 128; otherwise the CTA owns MB consecutive blocks.
    t.c_base = PAIR ? bx * (2 * MB * 128) + rank * 128 : bx * (MB * 128);
    t.r0 = by * R_CTA;
    t.grp = bz / sl;                        // which layer of the group
    t.z = z0 + bz - t.grp * sl;             // which token slice
    t.kb_begin = static_cast<int>(p.unit_begin[t.z]) * p.kb_unit;
    int kb_end = static_cast<int>(p.unit_begin[t.z + 1]) * p.kb_unit;
    if (kb_end > p.k_blocks) kb_end = p.k_blocks;
    t.kb_count = kb_end - t.kb_begin;
    return true;
  };

  if (threadIdx.x == 0) {
    s_abort = 0;
#pragma unroll
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&bar_full[s], FULL_ARRIVALS);
      ptx::mbar_init(&bar_empty[s], 1);
    }
    ptx::mbar_init(&bar_accum, 1);
    ptx::mbar_init(&bar_tmem_free, (kTcThreads / 32 - 2) * (PAIR ? 2 : 1));
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&maps.x[0]);
    ptx::prefetch_tensormap(&maps.a[0]);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(&s_tmem_base, 512);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(&s_tmem_base, 512);
      ptx::tmem_relinquish();
    }
  }
  ptx::fence_tc_before_sync();
  if (PAIR) ptx::cluster_sync_all(); else __syncthreads();
  ptx::fence_tc_after_sync();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  if (warp == 0) {
    // ================= TMA producer: one lane per slab =================
    const bool is_x = lane < X_SLABS;
    uint8_t* my_dst = tiles + lane * kTcSlabBytes;
    int s = 0, issued = 0;
    uint32_t ph = 0;
    bool alive = true;
    for (int k = 0; alive; ++k) {
      Tile t;
      if (!sched(k, t)) break;
      const CUtensorMap* map = is_x ? &maps.x[t.grp] : &maps.a[t.grp];
      int xcoord;
      if (is_x) {
        xcoord = t.c_base + (lane >> 1) * C_STEP + (lane & 1) * 64;
      } else if (PAIR) {
        // slab a of this CTA: 256-row chunk a/2 of the tile, this CTA's half of it
        const int a = lane - X_SLABS, q = a >> 1;
        const int wq = R_CTA - 256 * q < 256 ? R_CTA - 256 * q : 256;
        xcoord = t.r0 + 256 * q + rank * (wq >> 1) + (a & 1) * 64;
      } else {
        xcoord = t.r0 + (lane - X_SLABS) * 64;
      }
      int tok = t.kb_begin * kTcBK;
      int ready_upto = 0;        // COOP: chunks below this one are known to be complete
      const int chunk_end = (t.kb_begin + t.kb_count) * kTcBK / kCoopChunk +
                            (((t.kb_begin + t.kb_count) * kTcBK) % kCoopChunk != 0 ? 1 : 0);
      for (int it = 0; it < t.kb_count; ++it) {
        int ok = 1;
        if (COOP && tok / kCoopChunk >= ready_upto) {
          // The gather warps of the grid publish kCoopParts * coop_cg arrivals per chunk.  One
          // probe reads the counters of the next 32 chunks of this slice (lane l: chunk + l) and
          // advances ready_upto over the leading run of complete ones, so that a gather running
          // ahead costs the producer one L2 round trip per 32 chunks, not one per chunk.
          const int chunk = tok / kCoopChunk;
          const int* flags = p.coop_ctrl + kCoopCtrlInts + t.grp * p.coop_chunks;
          const int want = kCoopParts * p.coop_cg;
          const long long start = clock64();
          int n_ready = 0;
          while (true) {
            const int c = chunk + lane;
            const bool done = c < chunk_end && ptx::flag_load_acquire(flags + c) >= want;
            const uint32_t mask = __ballot_sync(0xffffffffu, done);
            n_ready = __ffs(~mask) - 1;            // leading run of complete chunks (mask != all ones
            if (mask == 0xffffffffu) n_ready = 32; // unless every lane saw a complete chunk)
            if (n_ready > 0) break;
            __nanosleep(32);
            int give_up = 0;
            if (lane == 0) give_up = (*abort_flag != 0 || clock64() - start > kTcWaitLimit) ? 1 : 0;
            if (__shfl_sync(0xffffffffu, give_up, 0)) break;
          }
          if (n_ready == 0) {
            if (lane == 0) {
              if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 500);
              *abort_flag = 1;
            }
            alive = false;
            break;
          }
          ready_upto = chunk + n_ready;
          __syncwarp();
          // generic-proxy stores of other SMs (acquired above) -> this warp's TMA reads
          ptx::fence_proxy_async_global();
        }
        if (lane == 0) {
          ok = ptx::mbar_wait_bounded(&bar_empty[s], ph ^ 1u, abort_flag, kTcWaitLimit) ? 1 : 0;
          if (ok) {
            // PAIR: the even CTA's barrier collects the bytes of both CTAs
            if (!PAIR) ptx::mbar_arrive_expect_tx(&bar_full[s], TMA_BYTES);
            else if (rank == 0) ptx::mbar_arrive_expect_tx(&bar_full[s], 2 * TMA_BYTES);
          } else {
            if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 100 + s);
            *abort_flag = 1;
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { alive = false; break; }
        if (lane < TMA_SLABS) {
          if (PAIR) ptx::tma_load_2d_pair(my_dst + s * STAGE_BYTES, map, xcoord, tok, &bar_full[s]);
          else ptx::tma_load_2d(my_dst + s * STAGE_BYTES, map, xcoord, tok, &bar_full[s]);
        }
        tok += kTcBK;
        ++issued;
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
    if (lane == 0 && *abort_flag != 0 && rank == 0) {
      // let the copies already issued land before the CTA gives its smem back
      const int first = issued > STAGES ? issued - STAGES : 0;
      for (int it = first; it < issued; ++it)
        ptx::mbar_wait_bounded(&bar_full[it % STAGES], static_cast<uint32_t>(it / STAGES) & 1u,
                               nullptr, kTcDrainLimit);
    }
  } else if (warp == 1) {
    // ================= MMA issuer: one thread (of the even CTA if PAIR) =================
    if (lane == 0 && rank == 0) {
      constexpr uint32_t LBO = kTcSlabBytes, SBO = 1024;
      const uint64_t desc0 = ptx::smem_desc_mn_sw128(ptx::smem_u32(tiles), LBO, SBO);
      bool ok = true;
      int s = 0;
      uint32_t ph = 0, tile_ph = 0;
      bool first_tile = true;
      for (int k = 0; ok; ++k) {
        Tile t;
        if (!sched(k, t)) break;
        if (!first_tile) {
          // the accumulators are reused: the epilogue warps (of both CTAs) must have read the
          // previous tile out of TMEM before the first MMA of this one overwrites it
          if (!ptx::mbar_wait_bounded(&bar_tmem_free, tile_ph ^ 1u, abort_flag, kTcWaitLimit)) {
            if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 250);
            *abort_flag = 1;
            ok = false;
            break;
          }
          ptx::fence_tc_after_sync();
        }
        first_tile = false;
        for (int it = 0; it < t.kb_count; ++it) {
          if (!ptx::mbar_wait_bounded(&bar_full[s], ph, abort_flag, kTcWaitLimit, 0, FUSED && PAIR)) {
            if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 200 + s);
            *abort_flag = 1;
            ok = false;
            break;
          }
          ptx::fence_tc_after_sync();
          const uint64_t dstage = desc0 + static_cast<uint64_t>((s * STAGE_BYTES) >> 4);
#pragma unroll
          for (int ks = 0; ks < kTcBK / 16; ++ks) {
            const uint32_t acc = (it | ks) != 0 ? 1u : 0u;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
              // 16 tokens = 2 groups of 8 rows = 2 * SBO bytes into every slab
              const uint64_t adesc = dstage + ((mb * 2 * kTcSlabBytes + ks * 2 * SBO) >> 4);
#pragma unroll
              for (int j = 0; j < R_CTA; j += 256) {
                constexpr int kFull = 256;
                const int ncols = R_CTA - j < kFull ? R_CTA - j : kFull;
                // slabs of this 256-row chunk in a CTA's stage: 4, or 2 when split over a pair
                const int bslab = PAIR ? (j / 256) * 2 : j / 64;
                const uint64_t bdesc =
                    dstage + ((X_SLABS * kTcSlabBytes + bslab * kTcSlabBytes + ks * 2 * SBO) >> 4);
                const uint32_t idesc = ptx::idesc_bf16_mn_mn(UMMA_M, static_cast<uint32_t>(ncols));
                const uint32_t d = tmem_base + static_cast<uint32_t>(mb * R_CTA + j);
                if (PAIR) ptx::mma_bf16_pair(d, adesc, bdesc, idesc, acc);
                else ptx::mma_bf16(d, adesc, bdesc, idesc, acc);
              }
            }
          }
          // frees the stage (in both CTAs if PAIR) once these MMAs have read it
          if (PAIR) ptx::mma_commit_pair(&bar_empty[s]); else ptx::mma_commit(&bar_empty[s]);
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        // accumulators of this tile complete (or: everything issued so far is done)
        if (PAIR) ptx::mma_commit_pair(&bar_accum); else ptx::mma_commit(&bar_accum);
        if (!ok) ptx::mbar_wait_bounded(&bar_accum, tile_ph, nullptr, kTcDrainLimit);
        tile_ph ^= 1u;
      }
    }
  } else if (COOP && warp >= kTcThreads / 32 && warp - kTcThreads / 32 < p.coop_warps) {
    // ================= gather warps (COOP): shared queue over the whole launch =================
    // Item = (token slice bz, chunk position pp in the slice, column group, part): one warp
    // copies dY[t, idx[j]] for the part's 16 tokens and up to 256 columns j into Ag[t, j].
    // Queue order follows the GEMM: slices grouped by the wave of tiles that first touches them,
    // inside a group chunk position first, so every running tile finds its next chunk early.
    // Padding items (a slice shorter than coop_pmax) are skipped.
    // Slices are taken in the order the schedule above starts them: the slices of each full
    // wave of long tiles, then one last group holding the slices first touched by the partly
    // filled long wave together with ALL short slices (the workers without a tile in that wave
    // start on the short tiles at the same moment).  Inside a group the chunk position runs
    // slowest, so every running tile finds its next chunk early.
    const int per_chunk = p.coop_cg * kCoopParts;
    const int full_waves = n_long / n_workers;
    const int bz_full = full_waves > 0 ? (full_waves * n_workers - 1) / txy + 1 : 0;  // slices of full waves
    const int cnt_long_last = p.groups * p.s_long - bz_full;      // long slices left for the last group
    const int cnt_last = cnt_long_last + p.groups * s_short;
    const int pmax_last = cnt_long_last > 0 && p.coop_pmax_long > p.coop_pmax_short ? p.coop_pmax_long
                                                                                    : p.coop_pmax_short;
    const int items_full = bz_full * p.coop_pmax_long * per_chunk;
    const int total = items_full + cnt_last * pmax_last * per_chunk;
    // The counter of a finished item is published from inside the next item (after its first
    // loads are issued), so that the fence's round trip does not sit between two batches of
    // loads.  (Popping the next item ahead of time as well was slower: an item popped early sits
    // idle while its chunk's other parts complete, and the consumers wait for the last part.)
    int* publish = nullptr;
    while (true) {
      int q = 0;
      if (lane == 0) q = atomicAdd(p.coop_ctrl, 1);
      q = __shfl_sync(0xffffffffu, q, 0);
      if (q >= total) break;
      int pp, z, grp, rem2;
      if (q < items_full) {
        // which full wave: its new slices are [bz_lo, bz_hi)
        int bz_lo = 0, bz_hi = 0, base = 0;
        for (int w = 0; w < full_waves; ++w) {
          bz_hi = ((w + 1) * n_workers - 1) / txy + 1;
          const int items = (bz_hi - bz_lo) * p.coop_pmax_long * per_chunk;
          if (q < base + items) break;
          base += items;
          bz_lo = bz_hi;
        }
        const int in_wave = q - base, cnt = bz_hi - bz_lo;
        pp = in_wave / (cnt * per_chunk);
        const int rem = in_wave - pp * (cnt * per_chunk);
        const int bz = bz_lo + rem / per_chunk;
        rem2 = rem - (rem / per_chunk) * per_chunk;
        grp = bz / p.s_long;
        z = bz - grp * p.s_long;
      } else {
        const int in_wave = q - items_full;
        pp = in_wave / (cnt_last * per_chunk);
        const int rem = in_wave - pp * (cnt_last * per_chunk);
        const int si = rem / per_chunk;
        rem2 = rem - si * per_chunk;
        if (si < cnt_long_last) {
          const int bz = bz_full + si;
          grp = bz / p.s_long;
          z = bz - grp * p.s_long;
        } else {
          const int bzs = si - cnt_long_last;
          grp = bzs / s_short;
          z = p.s_long + bzs - grp * s_short;
        }
      }
      const int cg = rem2 / kCoopParts, part = rem2 - cg * kCoopParts;
      const int chunk = static_cast<int>(p.unit_begin[z]) + pp;    // kb_unit blocks = one chunk
      if (chunk >= static_cast<int>(p.unit_begin[z + 1])) continue;   // padding item
      const int col0 = cg * kCoopCols;
      const int32_t* idx = p.idx[grp];
      int rows[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int j = col0 + 32 * i + lane;
        int row = -1;
        if (j < p.r) {
          row = __ldg(idx + j);
          if (row < 0 || row >= p.m) {
            record_status(p.status, GRASS_ERR_INVALID_ARG, row);
            row = -1;
          }
        }
        rows[i] = row;
      }
      const unsigned short* src = reinterpret_cast<const unsigned short*>(p.dY[grp]);
      unsigned short* dst = reinterpret_cast<unsigned short*>(p.Ag[grp]);
      const int tok0 = chunk * kCoopChunk + part;
      const int cols = p.r_pad - col0;
      if (cols <= 64) coop_gather_part<2>(src, p.lddy, dst, p.r_pad, col0, rows, tok0, p.T, lane, publish);
      else if (cols <= 128) coop_gather_part<4>(src, p.lddy, dst, p.r_pad, col0, rows, tok0, p.T, lane, publish);
      else coop_gather_part<8>(src, p.lddy, dst, p.r_pad, col0, rows, tok0, p.T, lane, publish);
      publish = p.coop_ctrl + kCoopCtrlInts + grp * p.coop_chunks + chunk;
    }
    if (publish != nullptr) {
      __syncwarp();
      if (lane == 0) ptx::flag_arrive_release(publish);
    }
  } else if (FUSED && warp >= kTcThreads / 32) {
    // ================= gather warps (FUSED): dY[t, idx[j]] -> swizzled B-operand slabs =================
    // Warp g takes tokens g, g + GW, ... of the stage; lane l carries j = slab base + l and + 32:
    // one load instruction reads 32 neighbouring selected columns of one dY row.  The bytes go
    // where a TMA box {64, BK} with the 128-byte swizzle would put them: row t of a slab is 128
    // bytes, its 16-byte chunks XOR-ed with (t mod 8).
    const int g = warp - kTcThreads / 32;
    constexpr int GW = kTcGatherThreads / 32;
    int s = 0;
    uint32_t ph = 0;
    bool alive = true;
    for (int k = 0; alive; ++k) {
      Tile t;
      if (!sched(k, t)) break;
      const unsigned short* src = reinterpret_cast<const unsigned short*>(p.dY[t.grp]);
      const int32_t* idx = p.idx[t.grp];
      int rows[A_SLABS][2];
#pragma unroll
      for (int a = 0; a < A_SLABS; ++a) {
        int jb;
        if (PAIR) {
          const int q2 = a >> 1;
          const int wq = R_CTA - 256 * q2 < 256 ? R_CTA - 256 * q2 : 256;
          jb = t.r0 + 256 * q2 + rank * (wq >> 1) + (a & 1) * 64;
        } else {
          jb = t.r0 + a * 64;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int j = jb + 32 * h + lane;
          int row = -1;
          if (j < p.r) {
            row = __ldg(idx + j);
            if (row < 0 || row >= p.m) {
              record_status(p.status, GRASS_ERR_INVALID_ARG, row);
              row = -1;
            }
          }
          rows[a][h] = row;
        }
      }
      int tok0 = t.kb_begin * kTcBK;
      for (int it = 0; it < t.kb_count; ++it) {
        int ok = 1;
        if (lane == 0)
          ok = ptx::mbar_wait_bounded(&bar_empty[s], ph ^ 1u, abort_flag, kTcWaitLimit) ? 1 : 0;
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) {
          if (lane == 0) {
            if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 400 + s);
            *abort_flag = 1;
          }
          alive = false;
          break;
        }
        uint8_t* stage = tiles + s * STAGE_BYTES + X_SLABS * kTcSlabBytes;
#pragma unroll
        for (int a = 0; a < A_SLABS; ++a) {
          // all loads of this warp's share of the slab first (kTcBK / GW tokens x 2 per lane in
          // flight), then the stores: the gather is latency-bound otherwise
          constexpr int NT = kTcBK / GW;
          unsigned short v0[NT], v1[NT];
#pragma unroll
          for (int k = 0; k < NT; ++k) {
            const int tok = tok0 + g + k * GW;
            const unsigned short* line = src + static_cast<long long>(tok) * p.lddy;
            v0[k] = 0;
            v1[k] = 0;
            if (tok < p.T) {
              if (rows[a][0] >= 0) v0[k] = __ldg(line + rows[a][0]);
              if (rows[a][1] >= 0) v1[k] = __ldg(line + rows[a][1]);
            }
          }
#pragma unroll
          for (int k = 0; k < NT; ++k) {
            const int tt = g + k * GW;
            uint8_t* rowp = stage + a * kTcSlabBytes + tt * 128;
            const int sw = tt & 7;
            *reinterpret_cast<unsigned short*>(rowp + (((lane >> 3) ^ sw) << 4) + (lane & 7) * 2) = v0[k];
            *reinterpret_cast<unsigned short*>(rowp + ((((lane >> 3) + 4) ^ sw) << 4) + (lane & 7) * 2) = v1[k];
          }
        }
        ptx::fence_proxy_async_smem();   // generic writes -> visible to the MMA's async proxy
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive_leader(&bar_full[s]);
        tok0 += kTcBK;
        if (++s == STAGES) { s = 0; ph ^= 1u; }
      }
    }
  } else {
    // ================= epilogue: TMEM -> registers -> global =================
    const int q = warp & 3;             // TMEM lane quarter this warp may touch
    const int half = (warp - 2) >> 2;   // which of the quarter's two warps
    uint32_t tile_ph = 0;
    bool alive = true;
    for (int k = 0; alive; ++k) {
      Tile t;
      if (!sched(k, t)) break;
      // one polling lane per warp, with back-off: this wait lasts a whole main loop
      int got = 1;
      if (lane == 0) {
        got = ptx::mbar_wait_bounded(&bar_accum, tile_ph, abort_flag, kTcWaitLimit, 128) ? 1 : 0;
        if (!got) {
          if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 300 + warp);
          *abort_flag = 1;
        }
      }
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got || *abort_flag != 0) { alive = false; break; }
      tile_ph ^= 1u;
      ptx::fence_tc_after_sync();
      float* out = p.out[t.grp] + static_cast<long long>(t.z) * p.split_stride;
      const float* rho = p.rho[t.grp];
      const bool scale = p.split_k == 1 && rho != nullptr;
      const long long ld = p.ld_out;
#pragma unroll 1
      for (int chunk = half; chunk < MB * (R_CTA / 32); chunk += 2) {
        const int mb = chunk / (R_CTA / 32);
        const int j = (chunk % (R_CTA / 32)) * 32;
        const int row0 = t.r0 + j;
        if (row0 >= p.r) continue;      // uniform: padding rows
        uint32_t v[32];
        ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                               static_cast<uint32_t>(mb * R_CTA + j), v);
        ptx::tmem_ld_wait();
        const int c = t.c_base + mb * C_STEP + q * 32 + lane;
        if (p.norm_part != nullptr) {
          // fused row norms of the dense gradient (columns past n were zero-filled by TMA)
          float sq[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) sq[i] = __uint_as_float(v[i]) * __uint_as_float(v[i]);
          const float total = warp_transpose_sum(sq, lane);
          const int g = (t.c_base + mb * C_STEP + q * 32) >> 5;
          if (row0 + lane < p.r && (g << 5) < p.n) p.norm_part[g * p.ld_norm + row0 + lane] = total;
          continue;
        }
        float my_rho = 1.f;
        if (scale && row0 + lane < p.r) my_rho = __ldg(rho + row0 + lane);
        float* dst = out + static_cast<long long>(row0) * ld + c;
        const int nvalid = p.r - row0 < 32 ? p.r - row0 : 32;
        if (nvalid == 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float val = __uint_as_float(v[i]) * __shfl_sync(0xffffffffu, my_rho, i);
            if (c < p.n) dst[i * ld] = val;
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float val = __uint_as_float(v[i]) * __shfl_sync(0xffffffffu, my_rho, i);
            if (c < p.n && i < nvalid) dst[i * ld] = val;
          }
        }
      }
      // this warp's reads of TMEM are complete (tcgen05.wait::ld above): tell the MMA issuer
      ptx::fence_tc_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive_leader(&bar_tmem_free);
    }
  }
  __syncwarp();
  ptx::fence_tc_before_sync();
  // PAIR: neither CTA may leave (or free TMEM) while the other can still read its shared
  // memory through the MMA or signal its barriers
  if (PAIR) ptx::cluster_sync_all(); else __syncthreads();
  if (warp == 1) {
    ptx::fence_tc_after_sync();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, 512); else ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Ag[t, j] = dY[t, idx[j]] (bf16 bits copied unchanged), zero for r <= j < r_pad.
// HBM moves at least 32-byte sectors (16 bf16), so the copy reads 2 T m (1 - (1 - r/m)^16)
// bytes of dY or more however it is written (practically all of dY from r/m = 1/16 up);
// what the kernel controls is how many sector look-ups the load unit performs per useful byte.
constexpr int kGatherThreads = 256;
constexpr int kGatherTokens = 32;            // tokens per block
struct GatherGroup {
  const __nv_bfloat16* dY[kTcMaxGroup];
  const int32_t* idx[kTcMaxGroup];
  __nv_bfloat16* Ag[kTcMaxGroup];
};

// A warp owns one token at a time and 32 * ni consecutive j: lane l loads
// j = jb + 32 i + l for i < ni, so one load instruction covers 32 neighbouring
// selected columns (ascending idx: as few 32-byte sectors as the selection
// allows) and one store instruction writes 64 contiguous bytes of Ag.
__global__ void __launch_bounds__(kGatherThreads)
gather_cols_kernel(const GatherGroup grp, long long lddy, int T, int m, int r, int r_pad, int ni,
                   int* status) {
  // blockIdx.z = layer of the group
  const __nv_bfloat16* __restrict__ dY = grp.dY[blockIdx.z];
  const int32_t* __restrict__ idx = grp.idx[blockIdx.z];
  __nv_bfloat16* __restrict__ Ag = grp.Ag[blockIdx.z];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int jb = blockIdx.x * (32 * ni);
  int rows[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int j = jb + 32 * i + lane;
    int row = -1;
    if (i < ni && j < r) {
      row = __ldg(idx + j);
      if (row < 0 || row >= m) {
        record_status(status, GRASS_ERR_INVALID_ARG, row);
        row = -1;
      }
    }
    rows[i] = row;
  }
  const unsigned short* src = reinterpret_cast<const unsigned short*>(dY);
  unsigned short* dst = reinterpret_cast<unsigned short*>(Ag);
  const int t_begin = blockIdx.y * kGatherTokens;
  const int t_end = t_begin + kGatherTokens < T ? t_begin + kGatherTokens : T;
#pragma unroll 2
  for (int t = t_begin + warp; t < t_end; t += kGatherThreads / 32) {
    const unsigned short* line = src + static_cast<long long>(t) * lddy;
    unsigned short v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = rows[i] >= 0 ? __ldg(line + rows[i]) : 0;
    unsigned short* out = dst + static_cast<long long>(t) * r_pad + jb + lane;
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if (i < ni && jb + 32 * i + lane < r_pad) out[32 * i] = v[i];
  }
}

struct ReduceGroup {
  const float* part[kTcMaxGroup];
  const float* rho[kTcMaxGroup];
  float* Gc[kTcMaxGroup];
};

// Gc[j, c] = rho_j * sum_s part[s][j][c], splits added in increasing s.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const ReduceGroup grp, long long ld_part, long long split_stride, int split_k,
                     int r, int n, long long ldgc, int vec) {
  // blockIdx.y = layer of the group
  const float* __restrict__ part = grp.part[blockIdx.y];
  const float* __restrict__ rho = grp.rho[blockIdx.y];
  float* __restrict__ Gc = grp.Gc[blockIdx.y];
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  if (vec) {
    const int nv = n / 4;
    const long long total = static_cast<long long>(r) * nv;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += stride) {
      const int row = static_cast<int>(i / nv), col = static_cast<int>(i - static_cast<long long>(row) * nv) * 4;
      const float* src = part + static_cast<long long>(row) * ld_part + col;
      float4 acc = *reinterpret_cast<const float4*>(src);
      int s = 1;
      for (; s + 3 < split_k; s += 4) {   // four loads in flight; the order of the adds is fixed
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          v[u] = *reinterpret_cast<const float4*>(src + (s + u) * split_stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w;
        }
      }
      for (; s < split_k; ++s) {
        const float4 v = *reinterpret_cast<const float4*>(src + s * split_stride);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      const float sc = rho != nullptr ? __ldg(rho + row) : 1.f;
      acc.x *= sc; acc.y *= sc; acc.z *= sc; acc.w *= sc;
      *reinterpret_cast<float4*>(Gc + static_cast<long long>(row) * ldgc + col) = acc;
    }
  } else {
    const long long total = static_cast<long long>(r) * n;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += stride) {
      const int row = static_cast<int>(i / n), col = static_cast<int>(i - static_cast<long long>(row) * n);
      const float* src = part + static_cast<long long>(row) * ld_part + col;
      float acc = *src;
      for (int s = 1; s < split_k; ++s) acc += src[s * split_stride];
      Gc[static_cast<long long>(row) * ldgc + col] = acc * (rho != nullptr ? __ldg(rho + row) : 1.f);
    }
  }
}

// Row norms from split-K partials of a small dense gradient: norms[j] = sqrt(sum_c (sum_s
// part[s][j][c])^2).  One CTA per row; splits added in increasing s (four loads in flight),
// columns by a fixed thread-strided order, then a shuffle tree and one shared-memory hop:
// bit-reproducible.
__global__ void __launch_bounds__(256)
splitk_rownorms_kernel(const float* __restrict__ part, long long ld_part, long long split_stride,
                       int split_k, int m, int n, float* __restrict__ norms) {
  __shared__ float s_part[8];
  const int j = blockIdx.x;
  const float* row = part + static_cast<long long>(j) * ld_part;
  float acc = 0.f;
  for (int c = threadIdx.x; c < n; c += 256) {
    const float* p = row + c;
    float g = 0.f;
    int s = 0;
    for (; s + 3 < split_k; s += 4) {
      const float a0 = p[(s + 0) * split_stride], a1 = p[(s + 1) * split_stride],
                  a2 = p[(s + 2) * split_stride], a3 = p[(s + 3) * split_stride];
      g = (((g + a0) + a1) + a2) + a3;
    }
    for (; s < split_k; ++s) g += p[s * split_stride];
    acc = fmaf(g, g, acc);
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = threadIdx.x < 8 ? s_part[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) norms[j] = sqrtf(v);
  }
}

// norms[j] = sqrt(sum over column groups g of part[g][j]), groups added in increasing g.
__global__ void __launch_bounds__(256)
norms_finalize_kernel(const float* __restrict__ part, long long ld, int groups, int m,
                      float* __restrict__ norms) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  float acc = 0.f;
  for (int g = 0; g < groups; ++g) acc += part[g * ld + j];
  norms[j] = sqrtf(acc);
}

}  // namespace grass
