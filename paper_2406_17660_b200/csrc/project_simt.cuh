// fp32 path of grass_project_grad: Gc[j,c] = rho_j * sum_t dY[t,idx_j] X[t,c]
// (Section 3.1 of the GRASS paper) with fp32 FMA on the CUDA cores.
//
// Used when the caller asks for "fp32 everywhere": tensor-core TF32 would drop
// 13 mantissa bits of every product, so this path keeps full fp32 products.
// A CTA owns a 64 (j) x 64 (c) output tile; 256 threads hold 4 x 4 outputs
// each; tokens are staged 16 at a time through shared memory, the dY columns
// being gathered by idx on the way in.  Small problems are split over the tokens
// (gridDim.z slices, partials summed in slice order by splitk_reduce_kernel) so
// that more than a handful of SMs work; results are bit-reproducible.
#pragma once

#include "common.cuh"

namespace grass {

constexpr int kSimtBJ = 64, kSimtBC = 64, kSimtBT = 16, kSimtThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
project_simt_kernel(const T* __restrict__ dY, int64_t lddy, const T* __restrict__ X, int64_t ldx,
                    int64_t Ttok, int64_t m, int64_t n, const int32_t* __restrict__ idx,
                    const float* __restrict__ rho, int r, float* __restrict__ Gc, int64_t ldgc,
                    int64_t tokens_per_split, int64_t split_stride, int* status) {
  __shared__ float sA[kSimtBT][kSimtBJ + 1];   // sA[t][j] = dY[t0+t, idx[j0+j]]
  __shared__ float sX[kSimtBT][kSimtBC + 1];
  __shared__ int sRow[kSimtBJ];
  const int tid = threadIdx.x;
  const int j0 = blockIdx.y * kSimtBJ;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * kSimtBC;
  if (tid < kSimtBJ) {
    int row = -1;
    const int j = j0 + tid;
    if (j < r) {
      row = idx != nullptr ? idx[j] : j;
      if (row < 0 || row >= m) {
        record_status(status, GRASS_ERR_INVALID_ARG, row);
        row = -1;
      }
    }
    sRow[tid] = row;
  }
  __syncthreads();
  const int tj = (tid / 16) * 4, tc = (tid % 16) * 4;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  // blockIdx.z owns a slice of the tokens; with more than one slice the output is that slice's
  // partial sum (rho applied later by the reduction), written at z * split_stride
  const int64_t t_lo = static_cast<int64_t>(blockIdx.z) * tokens_per_split;
  const int64_t t_hi = t_lo + tokens_per_split < Ttok ? t_lo + tokens_per_split : Ttok;
  Gc += static_cast<int64_t>(blockIdx.z) * split_stride;
  for (int64_t t0 = t_lo; t0 < t_hi; t0 += kSimtBT) {
    for (int e = tid; e < kSimtBT * kSimtBJ; e += kSimtThreads) {
      const int tt = e / kSimtBJ, jj = e % kSimtBJ;
      const int row = sRow[jj];
      const int64_t t = t0 + tt;
      sA[tt][jj] = (row >= 0 && t < t_hi) ? to_float(dY[t * lddy + row]) : 0.f;
    }
    for (int e = tid; e < kSimtBT * kSimtBC; e += kSimtThreads) {
      const int tt = e / kSimtBC, cc = e % kSimtBC;
      const int64_t t = t0 + tt, c = c0 + cc;
      sX[tt][cc] = (c < n && t < t_hi) ? to_float(X[t * ldx + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int tt = 0; tt < kSimtBT; ++tt) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sA[tt][tj + i]; b[i] = sX[tt][tc + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[i][k] = fmaf(a[i], b[k], acc[i][k]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int j = j0 + tj + i;
    if (j >= r) continue;
    const float s = (rho != nullptr && gridDim.z == 1) ? rho[j] : 1.f;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int64_t c = c0 + tc + k;
      if (c < n) Gc[static_cast<int64_t>(j) * ldgc + c] = s * acc[i][k];
    }
  }
}

}  // namespace grass
