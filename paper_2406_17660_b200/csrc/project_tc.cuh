// bf16 tensor-core path of grass_project_grad (Section 3.1 of the GRASS paper):
//   Gc[j, c] = rho_j * sum_t dY[t, idx_j] * X[t, c].
//
// The contraction runs over tokens (T = 32K..64K) while the output r x n is
// small, so the kernel is organised around one rule: read X once.  A CTA owns
// an output tile of (MB * 128) columns of n by r_cta selected rows with
// MB * r_cta <= 512, i.e. all 512 fp32 TMEM columns, and a slice of the tokens
// (split-K); every X element it loads meets all r_cta rows.
//
// Operand roles are swapped with respect to the formula so that neither input
// needs a transpose in HBM:  D^T[c, j] = sum_t X[t, c] * A[t, j]  with
//   A-operand = X tile      (M = 128 columns of n, MN-major: c contiguous)
//   B-operand = gathered dY (N = up to 256 selected rows, MN-major: j contiguous)
// Both are staged by TMA as slabs of [32 tokens][64 elements] with the 128-byte
// swizzle, which is the canonical MN-major UMMA layout.  TMEM lane = c, TMEM
// column = j, so the epilogue's tcgen05.ld hands each warp 32 consecutive c for
// one j per register: every store instruction writes 128 contiguous bytes.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA
// issuer, warps 2..5 = epilogue (warp w reads TMEM lanes 32*(w%4)..+31).
// Every mbarrier wait is bounded; on expiry the CTA records GRASS_ERR_TIMEOUT,
// drains what it has in flight (bounded again), frees its TMEM and returns.
#pragma once

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace grass {

constexpr int kTcBK = 32;                 // tokens per pipeline stage
constexpr int kTcSlabBytes = kTcBK * 128; // [32 tokens][64 bf16]
constexpr int kTcThreads = 192;
constexpr int kTcMaxStages = 8;
constexpr long long kTcWaitLimit = 2000000000LL;  // SM clocks (~1 s)
constexpr long long kTcDrainLimit = 200000000LL;  // give-up path: wait for work in flight

struct TcParams {
  int T, n, r;          // logical sizes
  int r_cta;            // selected rows per CTA, multiple of 64, <= 512
  int MB;               // 128-column blocks of n per CTA: 1, 2 or 4; MB * r_cta <= 512
  int stages;           // pipeline depth
  int k_blocks;         // ceil(T / 32)
  int split_k;          // gridDim.z
  float* out;           // split_k == 1: Gc, else partials [split][r][ld_out]
  long long ld_out;     // row pitch of out, elements
  long long split_stride;  // elements between partials of consecutive splits
  const float* rho;     // applied here only when split_k == 1 (may be NULL)
  int* status;
};

__global__ void __launch_bounds__(kTcThreads, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmA,
                  const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kTcMaxStages];
  __shared__ __align__(8) uint64_t bar_empty[kTcMaxStages];
  __shared__ __align__(8) uint64_t bar_accum;
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                              ~static_cast<uintptr_t>(1023));
  const int x_slabs = 2 * p.MB, a_slabs = p.r_cta / 64;
  const uint32_t stage_bytes = static_cast<uint32_t>((x_slabs + a_slabs) * kTcSlabBytes);

  const int c_tile0 = blockIdx.x * p.MB * 128;
  const int r0 = blockIdx.y * p.r_cta;
  // this CTA's token blocks: [kb_begin, kb_end)
  const int kb_per = p.k_blocks / p.split_k, kb_rem = p.k_blocks % p.split_k;
  const int z = blockIdx.z;
  const int kb_begin = z * kb_per + (z < kb_rem ? z : kb_rem);
  const int kb_count = kb_per + (z < kb_rem ? 1 : 0);

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(&bar_full[s], 1);
      ptx::mbar_init(&bar_empty[s], 1);
    }
    ptx::mbar_init(&bar_accum, 1);
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmX);
    ptx::prefetch_tensormap(&tmA);
  }
  if (warp == 1) {
    ptx::tmem_alloc(&s_tmem_base, 512);
    ptx::tmem_relinquish();
  }
  ptx::fence_tc_before_sync();
  __syncthreads();
  ptx::fence_tc_after_sync();
  const uint32_t tmem_base = s_tmem_base;
  volatile int* abort_flag = &s_abort;

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      int issued = 0;
      for (int it = 0; it < kb_count; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = static_cast<uint32_t>(it / p.stages) & 1u;
        if (!ptx::mbar_wait_bounded(&bar_empty[s], ph ^ 1u, abort_flag, kTcWaitLimit)) {
          if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 100 + s);
          *abort_flag = 1;
          break;
        }
        ptx::mbar_arrive_expect_tx(&bar_full[s], stage_bytes);
        uint8_t* dst = tiles + static_cast<size_t>(s) * stage_bytes;
        const int tok = (kb_begin + it) * kTcBK;
        for (int i = 0; i < x_slabs; ++i)
          ptx::tma_load_2d(dst + i * kTcSlabBytes, &tmX, c_tile0 + i * 64, tok, &bar_full[s]);
        dst += x_slabs * kTcSlabBytes;
        for (int i = 0; i < a_slabs; ++i)
          ptx::tma_load_2d(dst + i * kTcSlabBytes, &tmA, r0 + i * 64, tok, &bar_full[s]);
        issued = it + 1;
      }
      if (*abort_flag != 0) {
        // let the copies already issued land before the CTA gives its smem back
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int it = first; it < issued; ++it)
          ptx::mbar_wait_bounded(&bar_full[it % p.stages],
                                 static_cast<uint32_t>(it / p.stages) & 1u, nullptr,
                                 kTcDrainLimit);
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t tiles_addr = ptx::smem_u32(tiles);
      const uint32_t lbo = kTcSlabBytes, sbo = 1024;
      bool ok = true;
      for (int it = 0; it < kb_count && ok; ++it) {
        const int s = it % p.stages;
        const uint32_t ph = static_cast<uint32_t>(it / p.stages) & 1u;
        if (!ptx::mbar_wait_bounded(&bar_full[s], ph, abort_flag, kTcWaitLimit)) {
          if (*abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 200 + s);
          *abort_flag = 1;
          ok = false;
          break;
        }
        ptx::fence_tc_after_sync();
        const uint32_t xs = tiles_addr + static_cast<uint32_t>(s) * stage_bytes;
        const uint32_t as = xs + static_cast<uint32_t>(x_slabs * kTcSlabBytes);
#pragma unroll
        for (int ks = 0; ks < kTcBK / 16; ++ks) {
          const uint32_t koff = static_cast<uint32_t>(ks) * 2u * sbo;  // 16 tokens = 2 groups of 8
          const uint32_t acc = (it > 0 || ks > 0) ? 1u : 0u;
          for (int mb = 0; mb < p.MB; ++mb) {
            const uint64_t adesc = ptx::smem_desc_mn_sw128(
                xs + static_cast<uint32_t>(mb * 2 * kTcSlabBytes) + koff, lbo, sbo);
            for (int j = 0; j < p.r_cta; j += 256) {
              const int ncols = p.r_cta - j < 256 ? p.r_cta - j : 256;
              const uint64_t bdesc = ptx::smem_desc_mn_sw128(
                  as + static_cast<uint32_t>((j / 64) * kTcSlabBytes) + koff, lbo, sbo);
              ptx::mma_bf16(tmem_base + static_cast<uint32_t>(mb * p.r_cta + j), adesc, bdesc,
                            ptx::idesc_bf16_mn_mn(128, static_cast<uint32_t>(ncols)), acc);
            }
          }
        }
        ptx::mma_commit(&bar_empty[s]);  // frees the stage once these MMAs have read it
      }
      ptx::mma_commit(&bar_accum);       // accumulators complete (or: everything issued is done)
      if (!ok) ptx::mbar_wait_bounded(&bar_accum, 0, nullptr, kTcDrainLimit);
    }
  } else {
    // ================= epilogue: TMEM -> registers -> global =================
    const int q = warp & 3;  // TMEM lane quarter this warp may touch
    bool ok = kb_count > 0;
    if (ok && !ptx::mbar_wait_bounded(&bar_accum, 0, abort_flag, kTcWaitLimit)) {
      if (lane == 0 && *abort_flag == 0) record_status(p.status, GRASS_ERR_TIMEOUT, 300 + warp);
      *abort_flag = 1;
      ok = false;
    }
    if (ok && *abort_flag == 0) {
      ptx::fence_tc_after_sync();
      float* out = p.out + static_cast<long long>(z) * p.split_stride;
      for (int mb = 0; mb < p.MB; ++mb) {
        const int c = c_tile0 + mb * 128 + q * 32 + lane;
        for (int j = 0; j < p.r_cta; j += 32) {
          if (r0 + j >= p.r) break;  // uniform: rest of this tile is padding
          uint32_t v[32];
          ptx::tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) +
                                 static_cast<uint32_t>(mb * p.r_cta + j), v);
          ptx::tmem_ld_wait();
          if (c < p.n) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int row = r0 + j + i;
              if (row < p.r) {
                float val = __uint_as_float(v[i]);
                if (p.split_k == 1 && p.rho != nullptr) val *= __ldg(p.rho + row);
                out[static_cast<long long>(row) * p.ld_out + c] = val;
              }
            }
          }
        }
      }
    }
  }
  ptx::fence_tc_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::fence_tc_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Ag[t, j] = dY[t, idx[j]] (bf16 bits copied unchanged), zero for r <= j < r_pad.
// One thread carries 8 consecutive j for a run of tokens: gathered 2-byte loads
// from one dY row (ascending idx keeps them in few sectors), one 16-byte store.
constexpr int kGatherThreads = 256;
constexpr int kGatherTokens = 32;

__global__ void __launch_bounds__(kGatherThreads)
gather_cols_kernel(const __nv_bfloat16* __restrict__ dY, long long lddy, int T, int m,
                   const int32_t* __restrict__ idx, int r, int r_pad,
                   __nv_bfloat16* __restrict__ Ag, int* status) {
  const int jg = blockIdx.x * kGatherThreads + threadIdx.x;  // group of 8 selected rows
  if (jg * 8 >= r_pad) return;
  int rows[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int j = jg * 8 + i;
    int row = -1;
    if (j < r) {
      row = __ldg(idx + j);
      if (row < 0 || row >= m) {
        record_status(status, GRASS_ERR_INVALID_ARG, row);
        row = -1;
      }
    }
    rows[i] = row;
  }
  const unsigned short* src = reinterpret_cast<const unsigned short*>(dY);
  const int t_begin = blockIdx.y * kGatherTokens;
  const int t_end = t_begin + kGatherTokens < T ? t_begin + kGatherTokens : T;
#pragma unroll 4
  for (int t = t_begin; t < t_end; ++t) {
    const unsigned short* line = src + static_cast<long long>(t) * lddy;
    unsigned short v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = rows[i] >= 0 ? __ldg(line + rows[i]) : 0;
    uint4 pack;
    pack.x = v[0] | (static_cast<uint32_t>(v[1]) << 16);
    pack.y = v[2] | (static_cast<uint32_t>(v[3]) << 16);
    pack.z = v[4] | (static_cast<uint32_t>(v[5]) << 16);
    pack.w = v[6] | (static_cast<uint32_t>(v[7]) << 16);
    *reinterpret_cast<uint4*>(Ag + static_cast<long long>(t) * r_pad + jg * 8) = pack;
  }
}

// Gc[j, c] = rho_j * sum_s part[s][j][c], splits added in increasing s.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ part, long long ld_part, long long split_stride,
                     int split_k, int r, int n, const float* __restrict__ rho,
                     float* __restrict__ Gc, long long ldgc, int vec) {
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  if (vec) {
    const int nv = n / 4;
    const long long total = static_cast<long long>(r) * nv;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += stride) {
      const int row = static_cast<int>(i / nv), col = static_cast<int>(i - static_cast<long long>(row) * nv) * 4;
      const float* src = part + static_cast<long long>(row) * ld_part + col;
      float4 acc = *reinterpret_cast<const float4*>(src);
      for (int s = 1; s < split_k; ++s) {
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

}  // namespace grass
