// grass_row_norms: lambda_k = ||G[k,:]||_2 (Section 3.2 of the GRASS paper).
//
// HBM-bound streaming reduction: 4 m n bytes in (fp32 G), 4 m out.  A row is
// owned by TPR threads (32 = one warp for short rows ... 256 = one CTA for long
// ones, chosen so that a thread has at least 16 vector loads to issue); each thread issues independent 128-bit loads (eight in flight per
// loop trip) into separate fp32 accumulators, then a shuffle tree (and, for a
// CTA-wide row, one shared-memory hop) finishes the sum.
#include "common.cuh"

namespace grass {
namespace {

constexpr int kThreads = 256;

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  using type = float4;
  static __device__ __forceinline__ float sumsq(const float4& v) {
    return v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  using type = uint4;
  static __device__ __forceinline__ float sumsq(const uint4& v) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      s += f.x * f.x + f.y * f.y;
    }
    return s;
  }
};

template <typename T, int TPR, bool VEC>
__global__ void __launch_bounds__(kThreads)
row_norms_kernel(const T* __restrict__ G, int64_t m, int64_t n, int64_t ldg,
                 float* __restrict__ norms) {
  constexpr int ROWS = kThreads / TPR;
  const int lane_in_row = threadIdx.x % TPR;
  const int64_t row = static_cast<int64_t>(blockIdx.x) * ROWS + threadIdx.x / TPR;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  if (row < m) {
    const T* g = G + row * ldg;
    if (VEC) {
      using V = typename Vec<T>::type;
      constexpr int N = Vec<T>::N;
      const V* gv = reinterpret_cast<const V*>(g);
      const int64_t nv = n / N;
      int64_t i = lane_in_row;
      for (; i + 7 * TPR < nv; i += 8 * TPR) {
        V v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = __ldg(gv + i + u * TPR);
        acc0 += Vec<T>::sumsq(v[0]) + Vec<T>::sumsq(v[4]);
        acc1 += Vec<T>::sumsq(v[1]) + Vec<T>::sumsq(v[5]);
        acc2 += Vec<T>::sumsq(v[2]) + Vec<T>::sumsq(v[6]);
        acc3 += Vec<T>::sumsq(v[3]) + Vec<T>::sumsq(v[7]);
      }
      for (; i + 3 * TPR < nv; i += 4 * TPR) {
        V a = __ldg(gv + i), b = __ldg(gv + i + TPR), c = __ldg(gv + i + 2 * TPR),
          d = __ldg(gv + i + 3 * TPR);
        acc0 += Vec<T>::sumsq(a);
        acc1 += Vec<T>::sumsq(b);
        acc2 += Vec<T>::sumsq(c);
        acc3 += Vec<T>::sumsq(d);
      }
      for (; i < nv; i += TPR) acc0 += Vec<T>::sumsq(__ldg(gv + i));
      for (int64_t c = nv * N + lane_in_row; c < n; c += TPR) {
        float v = to_float(g[c]);
        acc1 += v * v;
      }
    } else {
      for (int64_t c = lane_in_row; c < n; c += TPR) {
        float v = to_float(g[c]);
        acc0 += v * v;
      }
    }
  }
  float s = warp_sum((acc0 + acc1) + (acc2 + acc3));
  if (TPR == 32) {
    if (lane_in_row == 0 && row < m) norms[row] = sqrtf(s);
  } else {
    __shared__ float part[kThreads / 32];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (lane_in_row == 0 && row < m) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < TPR / 32; ++w) v += part[(threadIdx.x >> 5) + w];
      norms[row] = sqrtf(v);
    }
  }
}

template <typename T>
int launch(const void* G, int64_t m, int64_t n, int64_t ldg, float* norms, cudaStream_t s) {
  const T* g = static_cast<const T*>(G);
  const bool vec = aligned_to(G, 16) && (ldg % Vec<T>::N) == 0;
  // threads per row: enough 128-bit loads per thread (>= 16) to keep eight in flight
  const int64_t nv = n / Vec<T>::N;
  const int tpr = nv >= 16 * 256 ? 256 : nv >= 16 * 128 ? 128 : nv >= 16 * 64 ? 64 : 32;
  const unsigned grid = static_cast<unsigned>((m + kThreads / tpr - 1) / (kThreads / tpr));
  ProfileScope prof(GRASS_K_ROW_NORMS, s);
#define GRASS_NORMS_CASE(TPR)                                                                   \
  if (tpr == TPR) {                                                                             \
    if (vec) row_norms_kernel<T, TPR, true><<<grid, kThreads, 0, s>>>(g, m, n, ldg, norms);     \
    else     row_norms_kernel<T, TPR, false><<<grid, kThreads, 0, s>>>(g, m, n, ldg, norms);    \
  }
  GRASS_NORMS_CASE(32) GRASS_NORMS_CASE(64) GRASS_NORMS_CASE(128) GRASS_NORMS_CASE(256)
#undef GRASS_NORMS_CASE
  GRASS_LAUNCH_CHECK();
  return GRASS_OK;
}

}  // namespace
}  // namespace grass

extern "C" int grass_row_norms(const void* G, int dt, int64_t m, int64_t n, int64_t ldg,
                               float* norms, void* stream) {
  if (G == nullptr || norms == nullptr || m < 1 || n < 1 || ldg < n || m > 0x7fffffffLL)
    return GRASS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dt == GRASS_F32) return grass::launch<float>(G, m, n, ldg, norms, s);
  if (dt == GRASS_BF16) return grass::launch<__nv_bfloat16>(G, m, n, ldg, norms, s);
  return GRASS_ERR_UNSUPPORTED;
}
