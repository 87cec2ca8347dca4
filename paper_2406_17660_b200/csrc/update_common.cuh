// Pieces shared by the Adam, apply and fused Adam+apply kernels.
#pragma once

#include <math.h>

#include "common.cuh"

namespace grass {

struct AdamScalars {
  float beta1, beta2, om_beta1, om_beta2, inv_bc1, inv_bc2, lr, eps;
};

// One element of adam.update.  Every rounding is spelled out (no compiler-chosen FMA
// contraction), so each kernel that inlines this produces the same bits.
__device__ __forceinline__ void adam_elem(float g, float& m, float& v, float& u,
                                          const AdamScalars& a) {
  m = __fmaf_rn(a.beta1, m, __fmul_rn(a.om_beta1, g));
  v = __fmaf_rn(a.beta2, v, __fmul_rn(a.om_beta2, __fmul_rn(g, g)));
  const float mhat = __fmul_rn(m, a.inv_bc1);
  const float vhat = __fmul_rn(v, a.inv_bc2);
  u = __fdiv_rn(__fmul_rn(-a.lr, mhat), __fadd_rn(__fsqrt_rn(vhat), a.eps));
}
// acc + s * u, one rounding: the accumulation of the apply step.
__device__ __forceinline__ float apply_acc(float acc, float s, float u) { return __fmaf_rn(s, u, acc); }

// Host: the fp32 scalars of one adam.update, formed in double (Appendix A of the paper).
inline AdamScalars make_adam_scalars(double lr, double beta1, double beta2, double eps, int step) {
  AdamScalars a;
  a.beta1 = static_cast<float>(beta1);
  a.beta2 = static_cast<float>(beta2);
  a.om_beta1 = static_cast<float>(1.0 - beta1);
  a.om_beta2 = static_cast<float>(1.0 - beta2);
  a.inv_bc1 = static_cast<float>(1.0 / (1.0 - pow(beta1, static_cast<double>(step))));
  a.inv_bc2 = static_cast<float>(1.0 / (1.0 - pow(beta2, static_cast<double>(step))));
  a.lr = static_cast<float>(lr);
  a.eps = static_cast<float>(eps);
  return a;
}
inline bool adam_args_ok(double lr, double beta1, double beta2, double eps, int step) {
  return step >= 1 && beta1 >= 0.0 && beta1 < 1.0 && beta2 >= 0.0 && beta2 < 1.0 && eps >= 0.0 &&
         isfinite(lr);
}

// Element type of W: vector width, load/add/round/store.
template <typename T> struct WTraits;
template <> struct WTraits<float> {
  static constexpr int N = 4;
  using vec = float4;
  static __device__ __forceinline__ void add_store(float* w, float4 v, const float* acc) {
    v.x += acc[0]; v.y += acc[1]; v.z += acc[2]; v.w += acc[3];
    *reinterpret_cast<float4*>(w) = v;
  }
  static __device__ __forceinline__ float add1(float w, float a) { return w + a; }
};
template <> struct WTraits<__nv_bfloat16> {
  static constexpr int N = 8;
  using vec = uint4;
  static __device__ __forceinline__ void add_store(__nv_bfloat16* w, uint4 raw, const float* acc) {
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      f.x += acc[2 * i];
      f.y += acc[2 * i + 1];
      h[i] = __floats2bfloat162_rn(f.x, f.y);
    }
    *reinterpret_cast<uint4*>(w) = raw;
  }
  static __device__ __forceinline__ __nv_bfloat16 add1(__nv_bfloat16 w, float a) {
    return __float2bfloat16_rn(__bfloat162float(w) + a);
  }
};

}  // namespace grass
