// grass_subspace_adam: adam.update on the r x n subspace state (Appendix A of
// the GRASS paper).
//
// HBM-bound elementwise kernel: reads g, M, V and writes M, V, U = 24 bytes per
// element, 128-bit accesses, no reuse.  The scalar factors (1 - beta, the
// reciprocal bias corrections) are formed in double on the host and rounded
// once to fp32.
#include "update_common.cuh"

namespace grass {
namespace {

constexpr int kThreads = 256;

// Vector path: n, ldgc, ldstate multiples of 4 and 16-byte aligned bases.
__global__ void __launch_bounds__(kThreads)
adam_vec4_kernel(const float* Gc, int64_t ldgc, float* __restrict__ M,
                 float* __restrict__ V, float* U, int64_t ldstate, int64_t nv, int64_t total,
                 AdamScalars a) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < total;
       i += stride) {
    const int64_t row = i / nv, col = (i - row * nv) * 4;
    const float4 g = *reinterpret_cast<const float4*>(Gc + row * ldgc + col);
    float4 m = *reinterpret_cast<float4*>(M + row * ldstate + col);
    float4 v = *reinterpret_cast<float4*>(V + row * ldstate + col);
    float4 u;
    adam_elem(g.x, m.x, v.x, u.x, a);
    adam_elem(g.y, m.y, v.y, u.y, a);
    adam_elem(g.z, m.z, v.z, u.z, a);
    adam_elem(g.w, m.w, v.w, u.w, a);
    *reinterpret_cast<float4*>(M + row * ldstate + col) = m;
    *reinterpret_cast<float4*>(V + row * ldstate + col) = v;
    *reinterpret_cast<float4*>(U + row * ldstate + col) = u;
  }
}

__global__ void __launch_bounds__(kThreads)
adam_scalar_kernel(const float* Gc, int64_t ldgc, float* __restrict__ M,
                   float* __restrict__ V, float* U, int64_t ldstate, int64_t n, int64_t total,
                   AdamScalars a) {
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kThreads + threadIdx.x; i < total;
       i += stride) {
    const int64_t row = i / n, col = i - row * n;
    const float g = Gc[row * ldgc + col];
    float m = M[row * ldstate + col], v = V[row * ldstate + col], u;
    adam_elem(g, m, v, u, a);
    M[row * ldstate + col] = m;
    V[row * ldstate + col] = v;
    U[row * ldstate + col] = u;
  }
}

}  // namespace
}  // namespace grass

extern "C" int grass_subspace_adam(const float* Gc, int64_t ldgc, float* M, float* V, float* U,
                                   int64_t ldstate, int32_t r, int64_t n, double lr,
                                   double beta1, double beta2, double eps, int32_t step,
                                   void* stream) {
  using namespace grass;
  if (Gc == nullptr || M == nullptr || V == nullptr || U == nullptr || r < 1 || n < 1 ||
      ldgc < n || ldstate < n || step < 1)
    return GRASS_ERR_INVALID_ARG;
  if (!adam_args_ok(lr, beta1, beta2, eps, step)) return GRASS_ERR_INVALID_ARG;
  const AdamScalars a = make_adam_scalars(lr, beta1, beta2, eps, step);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool vec = (n % 4 == 0) && (ldgc % 4 == 0) && (ldstate % 4 == 0) && aligned_to(Gc, 16) &&
                   aligned_to(M, 16) && aligned_to(V, 16) && aligned_to(U, 16);
  const int64_t max_blocks = 148LL * 16;
  ProfileScope prof(GRASS_K_ADAM, s);
  if (vec) {
    const int64_t nv = n / 4, total = static_cast<int64_t>(r) * nv;
    int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > max_blocks) blocks = max_blocks;
    adam_vec4_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, s>>>(Gc, ldgc, M, V, U, ldstate,
                                                                         nv, total, a);
  } else {
    const int64_t total = static_cast<int64_t>(r) * n;
    int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > max_blocks) blocks = max_blocks;
    adam_scalar_kernel<<<static_cast<unsigned>(blocks), kThreads, 0, s>>>(Gc, ldgc, M, V, U,
                                                                           ldstate, n, total, a);
  }
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}
