// Channel-wise gate (Eq. 4) on the tensor-core path.
//
// S(x, Delta, tau_c) switches an output channel off for an image when its gate fires at fewer
// than tau_c * h' * w' positions; a channel that is off takes Eq. 1's first case everywhere.  The
// decision needs every partial sum of the image, so the layer runs in two passes of the pixel-major
// tcgen05 kernel (tc_conv.cu):
//   1. base path and gate only (no conditional path): the mask of the plain gate;
//   2. counts per (image, channel) from that mask, and thresholds per (image, channel): the
//      layer's own where the channel stays on, +inf where it is off;
//   3. the whole layer with those thresholds.
// The counts are integers and the comparison with tau_c * h' * w' is the one the direct kernels
// and the oracle make, so the channel decisions agree whenever the gate decisions do.
#include "common.cuh"
#include "tc_conv.cuh"

namespace cg {
namespace {

size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// One block per (image, mask word): counts[n][32*w + b] = pixels of image n whose bit b of word w is set.
__global__ void __launch_bounds__(256) chan_count_kernel(const uint32_t* __restrict__ mask, int* __restrict__ counts,
                                                         int hw, int words, int c_out) {
  __shared__ int s_cnt[8][32];
  const int n = blockIdx.x / words, w = blockIdx.x - n * words;
  const int bit = threadIdx.x & 31, grp = threadIdx.x >> 5;
  int cnt = 0;
  for (int p = grp; p < hw; p += 8) cnt += (int)((mask[((size_t)n * hw + p) * words + w] >> bit) & 1u);
  s_cnt[grp][bit] = cnt;
  __syncthreads();
  if (grp == 0) {
    int total = 0;
#pragma unroll
    for (int g = 0; g < 8; ++g) total += s_cnt[g][bit];
    const int c = w * 32 + bit;
    if (c < c_out) counts[(size_t)n * c_out + c] = total;
  }
}

// Thresholds per (image, channel); counts the channels that are switched off and hands on an
// error that the first pass reported.
__global__ void __launch_bounds__(256) chan_decide_kernel(const int* __restrict__ counts, cg_bn_params bn,
                                                          const float* __restrict__ delta, float eps, int n, int c_out,
                                                          float need, float* __restrict__ t_img,
                                                          const unsigned long long* __restrict__ first_pass,
                                                          unsigned long long* __restrict__ counters) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i == 0 && first_pass[CNT_STATUS] != 0ull) {
    if (atomicCAS(&counters[CNT_STATUS], 0ull, first_pass[CNT_STATUS]) == 0ull)
      atomicExch(&counters[CNT_SITE], first_pass[CNT_SITE]);
  }
  if (i >= n * c_out) return;
  const int c = i % c_out;
  const bool on = (float)counts[i] >= need;            // theta(0) = 1: a count equal to the bound keeps the channel
  t_img[i] = on ? fold_channel(bn, delta, eps, c).t : __int_as_float(0x7f800000);
  if (!on) atomicAdd(&counters[CNT_CH_SKIPPED], 1ull);
}

}  // namespace

// [counts][thresholds][counters of the first pass][mask of the first pass][workspace of the kernel]
size_t tc_channel_gate_workspace_bytes(const LayerDims& L, const TcPlan& P) {
  return up256((size_t)L.n * L.c_out * 4) * 2 + 256 + up256((size_t)L.m * L.words * 4) + up256(tc_workspace_bytes(L, P));
}

int launch_tc_channel_gate(const LayerDims& L, const TcPlan& P, int in_dtype, TcMaps* maps, const void* x,
                           const void* w_base, const void* w_cond, const cg_bn_params& bn, const float* delta,
                           const void* residual, void* y, uint32_t* mask, void* workspace,
                           unsigned long long* counters, cudaStream_t stream) {
  if (!workspace) return (int)cudaErrorInvalidValue;
  char* ws = static_cast<char*>(workspace);
  const size_t nc = up256((size_t)L.n * L.c_out * 4);
  int* counts = reinterpret_cast<int*>(ws);
  float* t_img = reinterpret_cast<float*>(ws + nc);
  unsigned long long* first = reinterpret_cast<unsigned long long*>(ws + 2 * nc);
  uint32_t* mask1 = reinterpret_cast<uint32_t*>(ws + 2 * nc + 256);
  void* inner = ws + 2 * nc + 256 + up256((size_t)L.m * L.words * 4);
  if (cudaMemsetAsync(first, 0, 256, stream) != cudaSuccess) return (int)cudaErrorInvalidValue;
  int e = launch_tc(L, P, in_dtype, maps, x, w_base, w_cond, bn, delta, residual, y, mask1, inner, first, stream,
                    nullptr, 1);
  if (e != 0) return e;
  const int hw = L.ho * L.wo;
  chan_count_kernel<<<L.n * L.words, 256, 0, stream>>>(mask1, counts, hw, L.words, L.c_out);
  const float need = L.channel_tau * (float)hw;       // Eq. 4's bound on the count, in fp32 like the comparison
  chan_decide_kernel<<<(L.n * L.c_out + 255) / 256, 256, 0, stream>>>(counts, bn, delta, L.eps, L.n, L.c_out, need, t_img,
                                                                       first, counters);
  if (cudaGetLastError() != cudaSuccess) return (int)cudaErrorLaunchFailure;
  return launch_tc(L, P, in_dtype, maps, x, w_base, w_cond, bn, delta, residual, y, mask, inner, counters, stream,
                   t_img, 0);
}

}  // namespace cg
