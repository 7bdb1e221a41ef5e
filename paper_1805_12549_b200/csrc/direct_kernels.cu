// CUDA-core direct convolution of the channel-gated layer: the path for fp32 layers and for
// every shape the tensor-core path does not take.
//
// One warp owns one (pixel row m, 32-channel block q): lane = output channel.  Each lane runs
// the base-path sum (Section 3.1), takes the gate decision (Eq. 2/3), runs the conditional-path
// sum only if its own gate fired (Eq. 1), applies the path's batch norm and ReLU, and the
// warp's ballot is the mask word.  Floating-point sums run in the order (r, s, c_in) with
// separately rounded multiply and add, so results do not depend on the launch shape.
#include "common.cuh"
#include "direct_point.cuh"

namespace cg {
namespace {

__device__ __forceinline__ int conv_point_i8(const LayerDims& L, const int8_t* __restrict__ x,
                                             const int8_t* __restrict__ w, int n, int ho, int wo,
                                             int co, int c_lo, int cw) {
  int acc = 0;
  for (int r = 0; r < L.kh; ++r) {
    const int hi = ho * L.stride + r - L.pad;
    if (hi < 0 || hi >= L.h) continue;
    for (int s = 0; s < L.kw; ++s) {
      const int wi = wo * L.stride + s - L.pad;
      if (wi < 0 || wi >= L.w) continue;
      const int8_t* xp = x + (((long long)n * L.h + hi) * L.w + wi) * L.c_in + c_lo;
      const int8_t* wp = w + (((long long)co * L.kh + r) * L.kw + s) * cw;
      int ci = 0;
      // four products per instruction where both runs are 4-byte aligned (integer sums do not
      // depend on the order)
      if ((((uintptr_t)xp | (uintptr_t)wp) & 3u) == 0)
        for (; ci + 4 <= cw; ci += 4) acc = __dp4a(*(const int*)(xp + ci), *(const int*)(wp + ci), acc);
      for (; ci < cw; ++ci) acc += (int)xp[ci] * (int)wp[ci];
    }
  }
  return acc;
}

// Channel grouping (Section 3.3): the conditional path of output group g reads every input
// channel outside [g*c_p, (g+1)*c_p), in ascending order; weights are [c_out][kh][kw][c_r].
template <typename T>
__device__ __forceinline__ float conv_point_others(const LayerDims& L, const T* __restrict__ x,
                                                   const T* __restrict__ w, int n, int ho, int wo,
                                                   int co, int g) {
  float acc = 0.f;
  const int lo = g * L.c_p, hi2 = lo + L.c_p;
  for (int r = 0; r < L.kh; ++r) {
    const int hi = ho * L.stride + r - L.pad;
    if (hi < 0 || hi >= L.h) continue;
    for (int s = 0; s < L.kw; ++s) {
      const int wi = wo * L.stride + s - L.pad;
      if (wi < 0 || wi >= L.w) continue;
      const T* xp = x + (((long long)n * L.h + hi) * L.w + wi) * L.c_in;
      const T* wp = w + (((long long)co * L.kh + r) * L.kw + s) * L.c_r;
      for (int ci = 0; ci < lo; ++ci)
        acc = __fadd_rn(acc, __fmul_rn(Elem<T>::ld(xp + ci), Elem<T>::ld(wp + ci)));
      for (int ci = hi2; ci < L.c_in; ++ci)
        acc = __fadd_rn(acc, __fmul_rn(Elem<T>::ld(xp + ci), Elem<T>::ld(wp + ci - L.c_p)));
    }
  }
  return acc;
}

__device__ __forceinline__ int conv_point_others_i8(const LayerDims& L, const int8_t* __restrict__ x,
                                                    const int8_t* __restrict__ w, int n, int ho,
                                                    int wo, int co, int g) {
  int acc = 0;
  const int lo = g * L.c_p, hi2 = lo + L.c_p;
  for (int r = 0; r < L.kh; ++r) {
    const int hi = ho * L.stride + r - L.pad;
    if (hi < 0 || hi >= L.h) continue;
    for (int s = 0; s < L.kw; ++s) {
      const int wi = wo * L.stride + s - L.pad;
      if (wi < 0 || wi >= L.w) continue;
      const int8_t* xp = x + (((long long)n * L.h + hi) * L.w + wi) * L.c_in;
      const int8_t* wp = w + (((long long)co * L.kh + r) * L.kw + s) * L.c_r;
      for (int ci = 0; ci < lo; ++ci) acc += (int)xp[ci] * (int)wp[ci];
      for (int ci = hi2; ci < L.c_in; ++ci) acc += (int)xp[ci] * (int)wp[ci - L.c_p];
    }
  }
  return acc;
}

constexpr int kThreads = 256;

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads)
direct_gated_conv_kernel(LayerDims L, const TIn* __restrict__ x, const TIn* __restrict__ w_base,
                         const TIn* __restrict__ w_cond, cg_bn_params bn,
                         const float* __restrict__ delta, const TOut* __restrict__ residual,
                         TOut* __restrict__ y, uint32_t* __restrict__ mask,
                         float* __restrict__ p_out, int base_only,
                         unsigned long long* __restrict__ counters,
                         int chan_pass = 0, int* __restrict__ chan_cnt = nullptr, float chan_need = 0.f) {
  // chan_pass (channel-wise gate, Eq. 4): 1 = first pass: partial sums to p_out and, per image
  // and output channel, the number of firing gates to chan_cnt; 2 = second pass: partial sums
  // read back from p_out, conditional path only where the activation's gate fires AND the
  // channel's count reaches chan_need = tau_c * h' * w'.
  extern __shared__ float s_consts[];   // 6 * c_out: t, a1, b1, a2, b2, t2
  __shared__ unsigned long long s_active;
  float* s_t = s_consts;
  float* s_a1 = s_t + L.c_out;
  float* s_b1 = s_a1 + L.c_out;
  float* s_a2 = s_b1 + L.c_out;
  float* s_b2 = s_a2 + L.c_out;
  float* s_t2 = s_b2 + L.c_out;
  if (threadIdx.x == 0) s_active = 0ull;
  if (!base_only) {
    for (int c = threadIdx.x; c < L.c_out; c += blockDim.x) {
      const ChannelConsts k = fold_channel(bn, delta, L.eps, c);
      s_t[c] = k.t; s_a1[c] = k.a1; s_b1[c] = k.b1; s_a2[c] = k.a2; s_b2[c] = k.b2; s_t2[c] = k.t2;
    }
  }
  __syncthreads();

  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long items = L.m * L.words;
  unsigned long long my_active = 0;
  for (long long it = warp0; it < items; it += warps) {
    const long long m = it / L.words;
    const int q = (int)(it - m * L.words);
    const int co = q * 32 + lane;
    const bool valid = co < L.c_out;
    const int wo = (int)(m % L.wo);
    const int ho = (int)((m / L.wo) % L.ho);
    const int n = (int)(m / ((long long)L.wo * L.ho));
    bool fire = false;
    if (valid) {
      const int grp = L.grouping ? co / (L.c_out / L.groups) : 0;   // input group of the base path
      const float p = chan_pass == 2 ? p_out[m * L.c_out + co]
                                     : conv_point<TIn>(L, x, w_base, n, ho, wo, co, grp * L.c_p, L.c_p);
      if (base_only) {
        p_out[m * L.c_out + co] = p;
      } else if (chan_pass == 1) {
        p_out[m * L.c_out + co] = p;
        if (p >= s_t[co] && p <= s_t2[co]) atomicAdd(&chan_cnt[(long long)n * L.c_out + co], 1);
      } else {
        fire = (p >= s_t[co]) && (p <= s_t2[co]);   // NaN compares false; t2 = +inf unless the gate is two-sided
        if (chan_pass == 2) {
          const bool on = ((float)chan_cnt[(long long)n * L.c_out + co] >= chan_need);
          fire = fire && on;
          if (!on && ho == 0 && wo == 0) atomicAdd(&counters[CNT_CH_SKIPPED], 1ull);
        }
        float v;
        if (fire) {
          const float r = L.grouping ? conv_point_others<TIn>(L, x, w_cond, n, ho, wo, co, grp)
                                     : conv_point<TIn>(L, x, w_cond, n, ho, wo, co, L.c_p, L.c_r);
          v = __fadd_rn(__fmul_rn(s_a2[co], __fadd_rn(p, r)), s_b2[co]);
        } else {
          v = __fadd_rn(__fmul_rn(s_a1[co], p), s_b1[co]);
        }
        if (residual) v = __fadd_rn(v, (float)residual[m * L.c_out + co]);
        if (L.relu) v = (v > 0.f) ? v : 0.f;
        st_out(y + m * L.c_out + co, v);
      }
    }
    if (!base_only && chan_pass != 1) {
      const unsigned word = __ballot_sync(0xffffffffu, fire);
      if (lane == 0) {
        if (mask) mask[it] = word;
        my_active += __popc(word);
      }
    }
  }
  if (!base_only && chan_pass != 1) {
    if (lane == 0 && my_active) atomicAdd(&s_active, my_active);
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicAdd(&counters[CNT_CALLS], 1ull);
    if (threadIdx.x == 0 && s_active) {
      atomicAdd(&counters[CNT_ACTIVE], s_active);
    }
  }
}

__global__ void __launch_bounds__(kThreads)
direct_gated_conv_i8_kernel(LayerDims L, const int8_t* __restrict__ x,
                            const int8_t* __restrict__ w_base, const int8_t* __restrict__ w_cond,
                            cg_bn_params bn, int8_t* __restrict__ y, uint32_t* __restrict__ mask,
                            int* __restrict__ p_out, int base_only,
                            unsigned long long* __restrict__ counters) {
  __shared__ unsigned long long s_active;
  if (threadIdx.x == 0) s_active = 0ull;
  __syncthreads();
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long items = L.m * L.words;
  unsigned long long my_active = 0;
  for (long long it = warp0; it < items; it += warps) {
    const long long m = it / L.words;
    const int q = (int)(it - m * L.words);
    const int co = q * 32 + lane;
    const bool valid = co < L.c_out;
    const int wo = (int)(m % L.wo);
    const int ho = (int)((m / L.wo) % L.ho);
    const int n = (int)(m / ((long long)L.wo * L.ho));
    bool fire = false;
    if (valid) {
      const int grp = L.grouping ? co / (L.c_out / L.groups) : 0;
      const int p = conv_point_i8(L, x, w_base, n, ho, wo, co, grp * L.c_p, L.c_p);
      if (base_only) {
        p_out[m * L.c_out + co] = p;
      } else {
        fire = (p >= bn.q_gate_thr[co]);
        long long acc = p;
        if (fire) acc += L.grouping ? conv_point_others_i8(L, x, w_cond, n, ho, wo, co, grp)
                                    : conv_point_i8(L, x, w_cond, n, ho, wo, co, L.c_p, L.c_r);
        const bool full = fire;
        const long long mul = full ? bn.q_mul_full[co] : bn.q_mul_base[co];
        const long long off = full ? bn.q_off_full[co] : bn.q_off_base[co];
        long long qv = (acc * mul + off + (1ll << (L.shift - 1))) >> L.shift;
        const long long lo = L.relu ? 0 : -128;
        qv = qv < lo ? lo : (qv > 127 ? 127 : qv);
        y[m * L.c_out + co] = (int8_t)qv;
      }
    }
    if (!base_only) {
      const unsigned word = __ballot_sync(0xffffffffu, fire);
      if (lane == 0) {
        if (mask) mask[it] = word;
        my_active += __popc(word);
      }
    }
  }
  if (!base_only) {
    if (lane == 0 && my_active) atomicAdd(&s_active, my_active);
    __syncthreads();
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicAdd(&counters[CNT_CALLS], 1ull);
    if (threadIdx.x == 0 && s_active) {
      atomicAdd(&counters[CNT_ACTIVE], s_active);
    }
  }
}

}  // namespace

int launch_direct(const LayerDims& L, int in_dtype, const void* x, const void* w_base,
                  const void* w_cond, const cg_bn_params& bn, const float* delta,
                  const void* residual, void* y, uint32_t* mask, void* p_out, int base_only,
                  unsigned long long* counters, cudaStream_t stream) {
  const long long items = L.m * L.words;
  if (items == 0) return 0;
  const int warps_per_block = kThreads / 32;
  long long blocks = (items + warps_per_block - 1) / warps_per_block;
  const long long cap = 148ll * 8 * 8;
  if (blocks > cap) blocks = cap;
  const size_t smem = (size_t)6 * L.c_out * sizeof(float);
  if (in_dtype == CG_F32) {
    direct_gated_conv_kernel<float, float><<<(unsigned)blocks, kThreads, smem, stream>>>(
        L, (const float*)x, (const float*)w_base, (const float*)w_cond, bn, delta,
        (const float*)residual, (float*)y, mask, (float*)p_out, base_only, counters);
  } else if (in_dtype == CG_BF16) {
    direct_gated_conv_kernel<__nv_bfloat16, __nv_bfloat16><<<(unsigned)blocks, kThreads, smem, stream>>>(
        L, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_base, (const __nv_bfloat16*)w_cond, bn,
        delta, (const __nv_bfloat16*)residual, (__nv_bfloat16*)y, mask, (float*)p_out, base_only,
        counters);
  } else {
    direct_gated_conv_i8_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(
        L, (const int8_t*)x, (const int8_t*)w_base, (const int8_t*)w_cond, bn, (int8_t*)y, mask,
        (int*)p_out, base_only, counters);
  }
  return (int)cudaGetLastError();
}

// workspace of the channel-wise gate: [partial sums: M x c_out fp32][counts: n x c_out int32]
size_t channel_gate_workspace_bytes(const LayerDims& L) {
  const size_t p_bytes = ((size_t)L.m * L.c_out * sizeof(float) + 255) / 256 * 256;
  return p_bytes + ((size_t)L.n * L.c_out * sizeof(int) + 255) / 256 * 256;
}

int launch_direct_channel_gate(const LayerDims& L, int in_dtype, const void* x, const void* w_base,
                               const void* w_cond, const cg_bn_params& bn, const float* delta,
                               const void* residual, void* y, uint32_t* mask, void* workspace,
                               unsigned long long* counters, cudaStream_t stream) {
  const long long items = L.m * L.words;
  if (items == 0) return 0;
  if (in_dtype != CG_F32 && in_dtype != CG_BF16) return (int)cudaErrorInvalidValue;
  const size_t p_bytes = ((size_t)L.m * L.c_out * sizeof(float) + 255) / 256 * 256;
  float* p_ws = (float*)workspace;
  int* cnt_ws = (int*)((char*)workspace + p_bytes);
  cudaError_t e = cudaMemsetAsync(cnt_ws, 0, (size_t)L.n * L.c_out * sizeof(int), stream);
  if (e != cudaSuccess) return (int)e;
  const int warps_per_block = kThreads / 32;
  long long blocks = (items + warps_per_block - 1) / warps_per_block;
  const long long cap = 148ll * 8 * 8;
  if (blocks > cap) blocks = cap;
  const size_t smem = (size_t)6 * L.c_out * sizeof(float);
  // Eq. 4's threshold on the count, in fp32 like the comparison itself
  const float need = L.channel_tau * (float)(L.ho * L.wo);
  for (int pass = 1; pass <= 2; ++pass) {
    if (in_dtype == CG_F32) {
      direct_gated_conv_kernel<float, float><<<(unsigned)blocks, kThreads, smem, stream>>>(
          L, (const float*)x, (const float*)w_base, (const float*)w_cond, bn, delta,
          (const float*)residual, (float*)y, mask, p_ws, 0, counters, pass, cnt_ws, need);
    } else {
      direct_gated_conv_kernel<__nv_bfloat16, __nv_bfloat16><<<(unsigned)blocks, kThreads, smem, stream>>>(
          L, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_base, (const __nv_bfloat16*)w_cond, bn,
          delta, (const __nv_bfloat16*)residual, (__nv_bfloat16*)y, mask, p_ws, 0, counters, pass,
          cnt_ws, need);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
  }
  return 0;
}

}  // namespace cg
