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

constexpr int kMaxGroup = 8;

// Up to kMaxGroup same-shaped layers share one launch: blockIdx.z = layer of the group.
struct UpdateGroup {
  const float* Gc[kMaxGroup];
  float* M[kMaxGroup];
  float* V[kMaxGroup];
  float* U[kMaxGroup];
  void* W[kMaxGroup];
  const int32_t* idx[kMaxGroup];
  const float* rho[kMaxGroup];
};

template <typename T, bool VEC>
__global__ void __launch_bounds__(kThreads)
adam_scatter_kernel(const UpdateGroup grp, int64_t ldgc, int64_t ldstate, int64_t m, int64_t n,
                    int64_t ldw, int r, float alpha, AdamScalars a, int* status) {
  const float* __restrict__ Gc = grp.Gc[blockIdx.z];
  float* __restrict__ M = grp.M[blockIdx.z];
  float* __restrict__ V = grp.V[blockIdx.z];
  float* __restrict__ U = grp.U[blockIdx.z];
  T* __restrict__ W = static_cast<T*>(grp.W[blockIdx.z]);
  const int32_t* __restrict__ idx = grp.idx[blockIdx.z];
  const float* __restrict__ rho = grp.rho[blockIdx.z];
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
int launch(int count, const UpdateGroup& grp, int64_t ldgc, int64_t ldstate, int64_t m, int64_t n,
           int64_t ldw, int r, float alpha, const AdamScalars& a, cudaStream_t s) {
  constexpr int N = WTraits<T>::N;
  cudaError_t err;
  int* status = status_word(&err);
  if (status == nullptr) GRASS_CUDA_TRY(err);
  bool vec = (n % N == 0) && (ldw % N == 0) && (ldgc % 4 == 0) && (ldstate % 4 == 0);
  for (int g = 0; g < count; ++g)
    vec = vec && aligned_to(grp.W[g], 16) && aligned_to(grp.Gc[g], 16) && aligned_to(grp.M[g], 16) &&
          aligned_to(grp.V[g], 16) && (grp.U[g] == nullptr || aligned_to(grp.U[g], 16));
  dim3 grid(static_cast<unsigned>((n + kThreads * N - 1) / (kThreads * N)),
            static_cast<unsigned>(r), static_cast<unsigned>(count));
  ProfileScope prof(GRASS_K_ADAM_SCATTER, s);
  if (vec)
    adam_scatter_kernel<T, true><<<grid, kThreads, 0, s>>>(grp, ldgc, ldstate, m, n, ldw, r, alpha,
                                                           a, status);
  else
    adam_scatter_kernel<T, false><<<grid, kThreads, 0, s>>>(grp, ldgc, ldstate, m, n, ldw, r, alpha,
                                                            a, status);
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

int run(int count, const UpdateGroup& grp, int wdt, int64_t ldgc, int64_t ldstate, int64_t m,
        int64_t n, int64_t ldw, int r, double lr, double beta1, double beta2, double eps, int step,
        double alpha, cudaStream_t s) {
  if (m < 1 || n < 1 || r < 1 || r > 65535 || ldgc < n || ldstate < n || ldw < n ||
      m > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  for (int g = 0; g < count; ++g)
    if (grp.Gc[g] == nullptr || grp.M[g] == nullptr || grp.V[g] == nullptr ||
        grp.W[g] == nullptr || grp.idx[g] == nullptr)
      return GRASS_ERR_INVALID_ARG;
  if (!adam_args_ok(lr, beta1, beta2, eps, step)) return GRASS_ERR_INVALID_ARG;
  const AdamScalars a = make_adam_scalars(lr, beta1, beta2, eps, step);
  const float al = static_cast<float>(alpha);
  if (wdt == GRASS_F32)
    return launch<float>(count, grp, ldgc, ldstate, m, n, ldw, r, al, a, s);
  if (wdt == GRASS_BF16)
    return launch<__nv_bfloat16>(count, grp, ldgc, ldstate, m, n, ldw, r, al, a, s);
  return GRASS_ERR_UNSUPPORTED;
}

}  // namespace
}  // namespace grass

extern "C" int grass_adam_scatter(const float* Gc, int64_t ldgc, float* M, float* V, float* U,
                                  int64_t ldstate, void* W, int wdt, int64_t m, int64_t n,
                                  int64_t ldw, const int32_t* idx, const float* rho, int32_t r,
                                  double lr, double beta1, double beta2, double eps, int32_t step,
                                  double alpha, void* stream) {
  grass::UpdateGroup grp;
  for (int g = 0; g < grass::kMaxGroup; ++g) {
    grp.Gc[g] = Gc; grp.M[g] = M; grp.V[g] = V; grp.U[g] = U; grp.W[g] = W;
    grp.idx[g] = idx; grp.rho[g] = rho;
  }
  return grass::run(1, grp, wdt, ldgc, ldstate, m, n, ldw, r, lr, beta1, beta2, eps, step, alpha,
                    static_cast<cudaStream_t>(stream));
}

extern "C" int grass_adam_scatter_batched(int32_t count, const float* const* Gc, int64_t ldgc,
                                          float* const* M, float* const* V, float* const* U,
                                          int64_t ldstate, void* const* W, int wdt, int64_t m,
                                          int64_t n, int64_t ldw, const int32_t* const* idx,
                                          const float* const* rho, int32_t r, double lr,
                                          double beta1, double beta2, double eps, int32_t step,
                                          double alpha, void* stream) {
  if (count < 1 || count > grass::kMaxGroup || Gc == nullptr || M == nullptr || V == nullptr ||
      W == nullptr || idx == nullptr)
    return GRASS_ERR_INVALID_ARG;
  grass::UpdateGroup grp;
  for (int g = 0; g < grass::kMaxGroup; ++g) {
    const int gi = g < count ? g : 0;
    grp.Gc[g] = Gc[gi]; grp.M[g] = M[gi]; grp.V[g] = V[gi];
    grp.U[g] = U != nullptr ? U[gi] : nullptr;
    grp.W[g] = W[gi]; grp.idx[g] = idx[gi];
    grp.rho[g] = rho != nullptr ? rho[gi] : nullptr;
  }
  return grass::run(count, grp, wdt, ldgc, ldstate, m, n, ldw, r, lr, beta1, beta2, eps, step, alpha,
                    static_cast<cudaStream_t>(stream));
}
