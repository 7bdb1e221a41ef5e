// The ungated operators of a channel-gated ResNet-18 (cgnet.h): patch matrix of the stem,
// pixel subsampling for the 1x1 stride-2 shortcuts, max pooling, global average pooling.
// NHWC bf16; each is one memory-bound kernel that moves 16-byte vectors where the channel
// count allows.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cgnet.h"

namespace {

constexpr int kBlock = 256;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int grid_for(long long items, int cap = 148 * 16) {
  long long g = (items + kBlock - 1) / kBlock;
  if (g > cap) g = cap;
  if (g < 1) g = 1;
  return (int)g;
}

// One thread per group of eight consecutive columns of the patch matrix.
__global__ void __launch_bounds__(kBlock) im2col_kernel(const __nv_bfloat16* __restrict__ x,
                                                        __nv_bfloat16* __restrict__ a, int n, int h, int w,
                                                        int c, int k, int stride, int pad, int ho, int wo,
                                                        int k_pad) {
  const int vecs = k_pad >> 3;
  const long long total = (long long)n * ho * wo * vecs;
  const int kkc = k * k * c;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int v = (int)(i % vecs);
    long long m = i / vecs;
    const int j = (int)(m % wo); m /= wo;
    const int ii = (int)(m % ho);
    const int img = (int)(m / ho);
    __align__(16) __nv_bfloat16 out[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int col = v * 8 + e;
      __nv_bfloat16 val = __float2bfloat16(0.f);
      if (col < kkc) {
        const int ci = col % c, rs = col / c, s = rs % k, r = rs / k;
        const int yy = ii * stride + r - pad, xx = j * stride + s - pad;
        if (yy >= 0 && yy < h && xx >= 0 && xx < w) val = x[(((long long)img * h + yy) * w + xx) * c + ci];
      }
      out[e] = val;
    }
    *reinterpret_cast<uint4*>(a + i * 8) = *reinterpret_cast<const uint4*>(out);
  }
}

// The same for compile-time filter size, channel count and stride (the divisions become
// multiplications), one block per output row: the k input rows the output row reads are staged
// in shared memory once, then every thread gathers 16-byte vectors of the patch matrix from it.
template <int K, int C, int STRIDE>
__global__ void __launch_bounds__(kBlock) im2col_rows_kernel(const __nv_bfloat16* __restrict__ x,
                                                             __nv_bfloat16* __restrict__ a, int n, int h, int w,
                                                             int pad, int ho, int wo, int k_pad) {
  extern __shared__ __nv_bfloat16 rows[];               // [K][(w + 2*pad) * C], zero where outside the image
  const int row_len = (w + 2 * pad) * C;
  const int vecs = k_pad >> 3;
  constexpr int kkc = K * K * C;
  for (int job = blockIdx.x; job < n * ho; job += gridDim.x) {
    const int img = job / ho, i = job - img * ho;
    __syncthreads();                                    // the previous row's readers are done
    for (int t = threadIdx.x; t < K * row_len; t += blockDim.x) {
      const int r = t / row_len, q = t - r * row_len;
      const int yy = i * STRIDE + r - pad, xx = q / C - pad;
      __nv_bfloat16 v = __float2bfloat16(0.f);
      if (yy >= 0 && yy < h && xx >= 0 && xx < w) v = x[(((long long)img * h + yy) * w + xx) * C + (q % C)];
      rows[t] = v;
    }
    __syncthreads();
    __nv_bfloat16* out_row = a + (long long)job * wo * k_pad;
    for (int t = threadIdx.x; t < wo * vecs; t += blockDim.x) {
      const int j = t / vecs, v = t - j * vecs;
      __align__(16) __nv_bfloat16 out[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int col = v * 8 + e;
        // column (r, s, ci) reads the staged row r at pixel j*STRIDE + s (padding included), channel ci
        const int r = col / (K * C), sc = col - r * (K * C);
        out[e] = col < kkc ? rows[r * row_len + j * STRIDE * C + sc] : __float2bfloat16(0.f);
      }
      *reinterpret_cast<uint4*>(out_row + (long long)t * 8) = *reinterpret_cast<const uint4*>(out);
    }
  }
}

__global__ void __launch_bounds__(kBlock) subsample_kernel(const uint4* __restrict__ x, uint4* __restrict__ y,
                                                           int n, int h, int w, int cv, int stride, int ho,
                                                           int wo) {
  const long long total = (long long)n * ho * wo * cv;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int v = (int)(i % cv);
    long long m = i / cv;
    const int j = (int)(m % wo); m /= wo;
    const int ii = (int)(m % ho);
    const int img = (int)(m / ho);
    y[i] = x[(((long long)img * h + ii * stride) * w + j * stride) * cv + v];
  }
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a),
                                   *reinterpret_cast<const __nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}

__global__ void __launch_bounds__(kBlock) maxpool_kernel(const uint4* __restrict__ x, uint4* __restrict__ y,
                                                         int n, int h, int w, int cv, int k, int stride, int pad,
                                                         int ho, int wo) {
  const long long total = (long long)n * ho * wo * cv;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int v = (int)(i % cv);
    long long m = i / cv;
    const int j = (int)(m % wo); m /= wo;
    const int ii = (int)(m % ho);
    const int img = (int)(m / ho);
    const uint32_t ninf = 0xff80ff80u;   // two bf16 -inf
    uint4 best = make_uint4(ninf, ninf, ninf, ninf);
    for (int r = 0; r < k; ++r) {
      const int yy = ii * stride + r - pad;
      if (yy < 0 || yy >= h) continue;
      for (int s = 0; s < k; ++s) {
        const int xx = j * stride + s - pad;
        if (xx < 0 || xx >= w) continue;
        const uint4 t = x[(((long long)img * h + yy) * w + xx) * cv + v];
        best.x = max_bf16x2(best.x, t.x); best.y = max_bf16x2(best.y, t.y);
        best.z = max_bf16x2(best.z, t.z); best.w = max_bf16x2(best.w, t.w);
      }
    }
    y[i] = best;
  }
}

// One thread per (image, group of eight channels): fp32 sums over the pixels in order.
__global__ void __launch_bounds__(kBlock) avgpool_kernel(const uint4* __restrict__ x, uint4* __restrict__ y,
                                                         int n, int hw, int cv) {
  const int total = n * cv;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int v = i % cv, img = i / cv;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int p = 0; p < hw; ++p) {
      const uint4 t = x[((long long)img * hw + p) * cv + v];
      const __nv_bfloat16* tb = reinterpret_cast<const __nv_bfloat16*>(&t);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] += __bfloat162float(tb[e]);
    }
    __align__(16) __nv_bfloat16 out[8];
    const float inv = 1.0f / (float)hw;
#pragma unroll
    for (int e = 0; e < 8; ++e) out[e] = __float2bfloat16_rn(acc[e] * inv);
    y[i] = *reinterpret_cast<const uint4*>(out);
  }
}

cg_status launched() { return cudaGetLastError() == cudaSuccess ? CG_OK : CG_ERR_CUDA; }

}  // namespace

extern "C" {

cg_status cg_im2col_bf16(const void* x, void* a, int n, int h, int w, int c, int k, int stride, int pad,
                         int k_pad, void* cuda_stream) {
  if (!x || !a || n <= 0 || h <= 0 || w <= 0 || c <= 0 || k <= 0 || stride <= 0 || pad < 0) return CG_ERR_INVALID_ARG;
  if (k_pad < k * k * c || (k_pad & 7) || h + 2 * pad < k || w + 2 * pad < k) return CG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(a)) return CG_ERR_ALIGNMENT;
  const int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
  const long long items = (long long)n * ho * wo * (k_pad >> 3);
  const size_t stage = (size_t)k * (w + 2 * pad) * c * sizeof(__nv_bfloat16);
  if (k == 7 && c == 3 && stride == 2 && stage <= 48 * 1024) {   // the ResNet stem
    const int blocks = n * ho < 148 * 8 ? n * ho : 148 * 8;
    im2col_rows_kernel<7, 3, 2><<<blocks, kBlock, stage, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(a), n, h, w, pad, ho, wo, k_pad);
    return launched();
  }
  im2col_kernel<<<grid_for(items), kBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const __nv_bfloat16*>(x), static_cast<__nv_bfloat16*>(a), n, h, w, c, k, stride, pad, ho, wo, k_pad);
  return launched();
}

cg_status cg_subsample_bf16(const void* x, void* y, int n, int h, int w, int c, int stride, void* cuda_stream) {
  if (!x || !y || n <= 0 || h <= 0 || w <= 0 || c <= 0 || stride <= 0 || (c & 7)) return CG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y)) return CG_ERR_ALIGNMENT;
  const int ho = (h + stride - 1) / stride, wo = (w + stride - 1) / stride;
  const long long items = (long long)n * ho * wo * (c >> 3);
  subsample_kernel<<<grid_for(items), kBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(x), static_cast<uint4*>(y), n, h, w, c >> 3, stride, ho, wo);
  return launched();
}

cg_status cg_maxpool_bf16(const void* x, void* y, int n, int h, int w, int c, int k, int stride, int pad,
                          void* cuda_stream) {
  if (!x || !y || n <= 0 || h <= 0 || w <= 0 || c <= 0 || k <= 0 || stride <= 0 || pad < 0 || (c & 7)) return CG_ERR_INVALID_ARG;
  if (pad >= k || h + 2 * pad < k || w + 2 * pad < k) return CG_ERR_INVALID_ARG;   // every window holds a pixel
  if (!aligned16(x) || !aligned16(y)) return CG_ERR_ALIGNMENT;
  const int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
  const long long items = (long long)n * ho * wo * (c >> 3);
  maxpool_kernel<<<grid_for(items), kBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(x), static_cast<uint4*>(y), n, h, w, c >> 3, k, stride, pad, ho, wo);
  return launched();
}

cg_status cg_avgpool_bf16(const void* x, void* y, int n, int hw, int c, void* cuda_stream) {
  if (!x || !y || n <= 0 || hw <= 0 || c <= 0 || (c & 7)) return CG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y)) return CG_ERR_ALIGNMENT;
  avgpool_kernel<<<grid_for((long long)n * (c >> 3)), kBlock, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(x), static_cast<uint4*>(y), n, hw, c >> 3);
  return launched();
}

}  // extern "C"
