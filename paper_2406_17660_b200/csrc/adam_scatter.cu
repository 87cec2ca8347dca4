// grass_adam_scatter: adam.update on the subspace state (Appendix A of the GRASS
// paper) and the row-sparse apply W <- W + alpha P U (Algorithm 1) in one pass.
//
// The two steps are row-local: state row j and update row j feed only row
// idx[j] of W.  Running them back to back in one kernel keeps U in registers
// (it is written out only if the caller wants it), which removes the 8 bytes
// per element that the separate kernels spend writing and re-reading U, and
// one launch.  Per element: g 4 B in, M and V 4 B in + 4 B out each, W in +
// out.  The arithmetic is that of grass_subspace_adam followed by
// grass_scatter_update, operation for operation, so the results are
// bit-identical to calling the two.
//
// idx is ascending, so repeated rows are adjacent; the first j of a run owns
// the row of W, walks the run in order of j (updating each j's own state row)
// and writes the row once.
#include "update_common.cuh"

namespace grass {
namespace {

constexpr int kThreads = 256;

template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads)
adam_scatter_kernel(const float* __restrict__ Gc, int64_t ldgc, float* __restrict__ M,
                    float* __restrict__ V, float* __restrict__ U, int64_t ldstate,
                    T* __restrict__ W, int64_t m, int64_t n, int64_t ldw,
                    const int32_t* __restrict__ idx, const float* __restrict__ rho, int r,
                    float alpha, AdamScalars a, int* status) {
  const int j0 = blockIdx.y;
  const int row = idx[j0];
  if (j0 > 0 && idx[j0 - 1] == row) return;  // not the head of its run
  const bool valid = row >= 0 && row < m;
  if (!valid && threadIdx.x == 0 && blockIdx.x == 0)
    record_status(status, GRASS_ERR_INVALID_ARG, row);
  constexpr int N = WTraits<T>::N;
  if (VEC) {
    const int64_t c = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) * N;
    if (c >= n) return;
    float acc[N];
#pragma unroll
    for (int i = 0; i < N; ++i) acc[i] = 0.f;
    typename WTraits<T>::vec wv;
    T* w = W + static_cast<int64_t>(valid ? row : 0) * ldw + c;
    if (valid) wv = *reinterpret_cast<const typename WTraits<T>::vec*>(w);
    for (int j = j0; j < r && idx[j] == row; ++j) {
      const float s = alpha * (rho != nullptr ? rho[j] : 1.f);
      const int64_t so = static_cast<int64_t>(j) * ldstate + c;
      const float* g = Gc + static_cast<int64_t>(j) * ldgc + c;
#pragma unroll
      for (int q = 0; q < N / 4; ++q) {
        const float4 gv = __ldg(reinterpret_cast<const float4*>(g) + q);
        float4 mv = *(reinterpret_cast<float4*>(M + so) + q);
        float4 vv = *(reinterpret_cast<float4*>(V + so) + q);
        float4 uv;
        adam_elem(gv.x, mv.x, vv.x, uv.x, a);
        adam_elem(gv.y, mv.y, vv.y, uv.y, a);
        adam_elem(gv.z, mv.z, vv.z, uv.z, a);
        adam_elem(gv.w, mv.w, vv.w, uv.w, a);
        *(reinterpret_cast<float4*>(M + so) + q) = mv;
        *(reinterpret_cast<float4*>(V + so) + q) = vv;
        if (U != nullptr) *(reinterpret_cast<float4*>(U + so) + q) = uv;
        acc[4 * q + 0] = apply_acc(acc[4 * q + 0], s, uv.x);
        acc[4 * q + 1] = apply_acc(acc[4 * q + 1], s, uv.y);
        acc[4 * q + 2] = apply_acc(acc[4 * q + 2], s, uv.z);
        acc[4 * q + 3] = apply_acc(acc[4 * q + 3], s, uv.w);
      }
    }
    if (valid) WTraits<T>::add_store(w, wv, acc);
  } else {
    const int64_t c0 = (static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x) * N;
    for (int64_t c = c0; c < c0 + N && c < n; ++c) {
      float acc = 0.f;
      for (int j = j0; j < r && idx[j] == row; ++j) {
        const int64_t so = static_cast<int64_t>(j) * ldstate + c;
        float mv = M[so], vv = V[so], uv;
        adam_elem(Gc[static_cast<int64_t>(j) * ldgc + c], mv, vv, uv, a);
        M[so] = mv;
        V[so] = vv;
        if (U != nullptr) U[so] = uv;
        acc = apply_acc(acc, alpha * (rho != nullptr ? rho[j] : 1.f), uv);
      }
      if (valid) {
        T* w = W + static_cast<int64_t>(row) * ldw + c;
        *w = WTraits<T>::add1(*w, acc);
      }
    }
  }
}

template <typename T>
int launch(const float* Gc, int64_t ldgc, float* M, float* V, float* U, int64_t ldstate, void* W,
           int64_t m, int64_t n, int64_t ldw, const int32_t* idx, const float* rho, int r,
           float alpha, const AdamScalars& a, cudaStream_t s) {
  constexpr int N = WTraits<T>::N;
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  const bool vec = (n % N == 0) && (ldw % N == 0) && (ldgc % 4 == 0) && (ldstate % 4 == 0) &&
                   aligned_to(W, 16) && aligned_to(Gc, 16) && aligned_to(M, 16) &&
                   aligned_to(V, 16) && (U == nullptr || aligned_to(U, 16));
  dim3 grid(static_cast<unsigned>((n + kThreads * N - 1) / (kThreads * N)),
            static_cast<unsigned>(r));
  ProfileScope prof(GRASS_K_ADAM_SCATTER, s);
  if (vec)
    adam_scatter_kernel<T, true><<<grid, kThreads, 0, s>>>(Gc, ldgc, M, V, U, ldstate,
                                                           static_cast<T*>(W), m, n, ldw, idx, rho,
                                                           r, alpha, a, status);
  else
    adam_scatter_kernel<T, false><<<grid, kThreads, 0, s>>>(Gc, ldgc, M, V, U, ldstate,
                                                            static_cast<T*>(W), m, n, ldw, idx, rho,
                                                            r, alpha, a, status);
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

}  // namespace
}  // namespace grass

extern "C" int grass_adam_scatter(const float* Gc, int64_t ldgc, float* M, float* V, float* U,
                                  int64_t ldstate, void* W, int wdt, int64_t m, int64_t n,
                                  int64_t ldw, const int32_t* idx, const float* rho, int32_t r,
                                  double lr, double beta1, double beta2, double eps, int32_t step,
                                  double alpha, void* stream) {
  using namespace grass;
  if (Gc == nullptr || M == nullptr || V == nullptr || W == nullptr || idx == nullptr || m < 1 ||
      n < 1 || r < 1 || r > 65535 || ldgc < n || ldstate < n || ldw < n || m > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  if (!adam_args_ok(lr, beta1, beta2, eps, step)) return GRASS_ERR_INVALID_ARG;
  const AdamScalars a = make_adam_scalars(lr, beta1, beta2, eps, step);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const float al = static_cast<float>(alpha);
  if (wdt == GRASS_F32)
    return launch<float>(Gc, ldgc, M, V, U, ldstate, W, m, n, ldw, idx, rho, r, al, a, s);
  if (wdt == GRASS_BF16)
    return launch<__nv_bfloat16>(Gc, ldgc, M, V, U, ldstate, W, m, n, ldw, idx, rho, r, al, a, s);
  return GRASS_ERR_UNSUPPORTED;
}
