// grass_scatter_update: W <- W + alpha P U on the r selected rows only
// (Algorithm 1 "Apply update"; Section 3.1 "Efficient Weight Update").
//
// HBM-bound: per selected element 4 bytes of U in, one W element in and out.
// idx is ascending, so repeated rows are adjacent.  The first j of each run of
// equal rows owns the row: it sums alpha*rho_j*U[j,:] over its run in fp32, in
// order of j, and writes the row once -- no atomics, bit-reproducible.
#include "update_common.cuh"

namespace grass {
namespace {

constexpr int kThreads = 256;

template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads)
scatter_kernel(T* __restrict__ W, int64_t m, int64_t n, int64_t ldw, const float* __restrict__ U,
               int64_t ldu, const int32_t* __restrict__ idx, const float* __restrict__ rho, int r,
               float alpha, int* status) {
  const int j0 = blockIdx.y;
  const int row = idx[j0];
  if (j0 > 0 && idx[j0 - 1] == row) return;  // not the head of its run
  if (row < 0 || row >= m) {
    if (threadIdx.x == 0 && blockIdx.x == 0) record_status(status, GRASS_ERR_INVALID_ARG, row);
    return;
  }
  constexpr int N = WTraits<T>::N;
  T* w = W + static_cast<int64_t>(row) * ldw;
  if (VEC) {
    // two column chunks per thread, all loads of both issued before any arithmetic
    const int64_t ca = (static_cast<int64_t>(blockIdx.x) * 2 * kThreads + threadIdx.x) * N;
    const int64_t cb = ca + static_cast<int64_t>(kThreads) * N;
    if (ca >= n) return;
    const bool two = cb < n;
    float acc[2][N];
#pragma unroll
    for (int i = 0; i < N; ++i) acc[0][i] = acc[1][i] = 0.f;
    typename WTraits<T>::vec wa = *reinterpret_cast<const typename WTraits<T>::vec*>(w + ca), wb;
    if (two) wb = *reinterpret_cast<const typename WTraits<T>::vec*>(w + cb);
    for (int j = j0; j < r && idx[j] == row; ++j) {
      const float s = alpha * (rho != nullptr ? rho[j] : 1.f);
      const float* urow = U + static_cast<int64_t>(j) * ldu;
      float4 va[N / 4], vb[N / 4];
#pragma unroll
      for (int q = 0; q < N / 4; ++q) {
        va[q] = __ldg(reinterpret_cast<const float4*>(urow + ca) + q);
        if (two) vb[q] = __ldg(reinterpret_cast<const float4*>(urow + cb) + q);
      }
#pragma unroll
      for (int q = 0; q < N / 4; ++q) {
        acc[0][4 * q + 0] = apply_acc(acc[0][4 * q + 0], s, va[q].x); acc[0][4 * q + 1] = apply_acc(acc[0][4 * q + 1], s, va[q].y);
        acc[0][4 * q + 2] = apply_acc(acc[0][4 * q + 2], s, va[q].z); acc[0][4 * q + 3] = apply_acc(acc[0][4 * q + 3], s, va[q].w);
        if (two) {
          acc[1][4 * q + 0] = apply_acc(acc[1][4 * q + 0], s, vb[q].x); acc[1][4 * q + 1] = apply_acc(acc[1][4 * q + 1], s, vb[q].y);
          acc[1][4 * q + 2] = apply_acc(acc[1][4 * q + 2], s, vb[q].z); acc[1][4 * q + 3] = apply_acc(acc[1][4 * q + 3], s, vb[q].w);
        }
      }
    }
    WTraits<T>::add_store(w + ca, wa, acc[0]);
    if (two) WTraits<T>::add_store(w + cb, wb, acc[1]);
  } else {
    const int64_t c0 = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) * N;
    for (int64_t c = c0; c < c0 + N && c < n; ++c) {
      float acc = 0.f;
      for (int j = j0; j < r && idx[j] == row; ++j)
        acc = apply_acc(acc, alpha * (rho != nullptr ? rho[j] : 1.f), U[static_cast<int64_t>(j) * ldu + c]);
      w[c] = WTraits<T>::add1(w[c], acc);
    }
  }
}

// Column form (projection on the input dimension): W[c, idx_j] += alpha * rho_j * U[j, c].
// A block owns 32 rows c of W and 32 consecutive j.  The U tile is read with c contiguous,
// scaled, and transposed through shared memory; then lane l of a warp owns j = j0 + l, so the
// 32 lanes touch 32 ascending columns of one W row (few sectors).  The first j of a run of
// equal columns owns the column and adds the whole run (reaching past the tile through global
// memory if the run does), so every element is rounded once.
template <typename T>
__global__ void __launch_bounds__(kThreads)
scatter_cols_kernel(T* __restrict__ W, int64_t m, int64_t n, int64_t ldw,
                    const float* __restrict__ U, int64_t ldu, const int32_t* __restrict__ idx,
                    const float* __restrict__ rho, int r, float alpha, int* status) {
  __shared__ float tile[32][33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * 32;
  const int j0 = blockIdx.y * 32;
  for (int jj = warp; jj < 32; jj += kThreads / 32) {
    const int j = j0 + jj;
    float v = 0.f;
    if (j < r && c0 + lane < m)
      v = alpha * (rho != nullptr ? rho[j] : 1.f) * U[static_cast<int64_t>(j) * ldu + c0 + lane];
    tile[jj][lane] = v;
  }
  __syncthreads();
  const int j = j0 + lane;
  if (j >= r) return;
  const int col = idx[j];
  if (j > 0 && idx[j - 1] == col) return;              // not the head of its run
  if (col < 0 || col >= n) {
    if (blockIdx.x == 0 && warp == 0) record_status(status, GRASS_ERR_INVALID_ARG, col);
    return;
  }
  int run = 1;
  while (j + run < r && idx[j + run] == col) ++run;
  for (int cc = warp; cc < 32; cc += kThreads / 32) {
    const int64_t c = c0 + cc;
    if (c >= m) break;
    float acc = 0.f;
    for (int k = 0; k < run; ++k) {
      if (lane + k < 32) acc += tile[lane + k][cc];
      else acc += alpha * (rho != nullptr ? rho[j + k] : 1.f) * U[static_cast<int64_t>(j + k) * ldu + c];
    }
    T* w = W + c * ldw + col;
    *w = WTraits<T>::add1(*w, acc);
  }
}

template <typename T>
int launch(void* W, int64_t m, int64_t n, int64_t ldw, const float* U, int64_t ldu,
           const int32_t* idx, const float* rho, int r, float alpha, cudaStream_t s) {
  constexpr int N = WTraits<T>::N;
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  const bool vec = (n % N == 0) && (ldw % N == 0) && (ldu % 4 == 0) && aligned_to(W, 16) &&
                   aligned_to(U, 16);
  // vector path: a thread covers two chunks of N columns; scalar path: one
  const int64_t per_block = static_cast<int64_t>(kThreads) * N * (vec ? 2 : 1);
  dim3 grid(static_cast<unsigned>((n + per_block - 1) / per_block), static_cast<unsigned>(r));
  ProfileScope prof(GRASS_K_SCATTER, s);
  if (vec)
    scatter_kernel<T, true><<<grid, kThreads, 0, s>>>(static_cast<T*>(W), m, n, ldw, U, ldu, idx,
                                                      rho, r, alpha, status);
  else
    scatter_kernel<T, false><<<grid, kThreads, 0, s>>>(static_cast<T*>(W), m, n, ldw, U, ldu, idx,
                                                       rho, r, alpha, status);
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

}  // namespace
}  // namespace grass

extern "C" int grass_scatter_update(void* W, int wdt, int64_t m, int64_t n, int64_t ldw,
                                    const float* U, int64_t ldu, const int32_t* idx,
                                    const float* rho, int32_t r, double alpha, void* stream) {
  if (W == nullptr || U == nullptr || idx == nullptr || m < 1 || n < 1 || r < 1 || ldw < n ||
      ldu < n || r > 65535 || m > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const float a = static_cast<float>(alpha);
  if (wdt == GRASS_F32) return grass::launch<float>(W, m, n, ldw, U, ldu, idx, rho, r, a, s);
  if (wdt == GRASS_BF16)
    return grass::launch<__nv_bfloat16>(W, m, n, ldw, U, ldu, idx, rho, r, a, s);
  return GRASS_ERR_UNSUPPORTED;
}

extern "C" int grass_scatter_update_cols(void* W, int wdt, int64_t m, int64_t n, int64_t ldw,
                                         const float* U, int64_t ldu, const int32_t* idx,
                                         const float* rho, int32_t r, double alpha, void* stream) {
  using namespace grass;
  if (W == nullptr || U == nullptr || idx == nullptr || m < 1 || n < 1 || r < 1 || ldw < n ||
      ldu < m || r > 65535 * 32 || n > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  if (wdt != GRASS_F32 && wdt != GRASS_BF16) return GRASS_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  dim3 grid(static_cast<unsigned>((m + 31) / 32), static_cast<unsigned>((r + 31) / 32));
  const float a = static_cast<float>(alpha);
  ProfileScope prof(GRASS_K_SCATTER, s);
  if (wdt == GRASS_F32)
    scatter_cols_kernel<float><<<grid, kThreads, 0, s>>>(static_cast<float*>(W), m, n, ldw, U, ldu,
                                                         idx, rho, r, a, status);
  else
    scatter_cols_kernel<__nv_bfloat16><<<grid, kThreads, 0, s>>>(
        static_cast<__nv_bfloat16*>(W), m, n, ldw, U, ldu, idx, rho, r, a, status);
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}
