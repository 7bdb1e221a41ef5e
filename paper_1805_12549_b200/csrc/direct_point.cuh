// Direct-convolution building blocks shared by the CUDA-core kernels (direct_kernels.cu and
// noalloc.cu): element loads and stores, and the sum of one output activation over filter taps
// and a range of input channels, in the order (r, s, c_in) with separately rounded multiply and
// add (Section 3.1: the base-path and the conditional-path sums are this with different ranges).
#pragma once

#include "common.cuh"

namespace cg {

template <typename T> struct Elem;
template <> struct Elem<float> {
  static __device__ __forceinline__ float ld(const float* p) { return *p; }
};
template <> struct Elem<__nv_bfloat16> {
  static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

__device__ __forceinline__ void st_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void st_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Sum over taps and channels [c_lo, c_lo + cw) of one output activation.
template <typename T>
__device__ __forceinline__ float conv_point(const LayerDims& L, const T* __restrict__ x,
                                            const T* __restrict__ w, int n, int ho, int wo, int co,
                                            int c_lo, int cw) {
  float acc = 0.f;
  for (int r = 0; r < L.kh; ++r) {
    const int hi = ho * L.stride + r - L.pad;
    if (hi < 0 || hi >= L.h) continue;
    for (int s = 0; s < L.kw; ++s) {
      const int wi = wo * L.stride + s - L.pad;
      if (wi < 0 || wi >= L.w) continue;
      const T* xp = x + (((long long)n * L.h + hi) * L.w + wi) * L.c_in + c_lo;
      const T* wp = w + (((long long)co * L.kh + r) * L.kw + s) * cw;
      for (int ci = 0; ci < cw; ++ci)
        acc = __fadd_rn(acc, __fmul_rn(Elem<T>::ld(xp + ci), Elem<T>::ld(wp + ci)));
    }
  }
  return acc;
}

}  // namespace cg
