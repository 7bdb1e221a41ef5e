// cg_conv_forward_static: the gated layer for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the point where they run a layer: code
// running inside a memory pool that owns the whole device, a real-time loop that forbids calls
// which may synchronise the device, a plug-in that is handed tensors but no allocator.  The
// regular API needs a handle, and creating a handle allocates a counter block.  This entry
// point needs neither: its scratch (activity counters plus the per-channel gate/batch-norm
// constants, folded once per call by a small prologue kernel) lives in a file-scope device
// array that every GPU loading the library holds until the process exits.
//
// The layer itself runs on the CUDA-core direct path (any shape, floating-point dtypes), with
// the same arithmetic and summation order as cg_conv_forward with CG_ALGO_DIRECT.
#include <cstring>

#include "common.cuh"
#include "direct_point.cuh"

namespace cg {
namespace {

constexpr int kMaxChannels = CG_STATIC_MAX_C_OUT;
constexpr int kCounterBytes = 256;                       // CNT_SLOTS x u64, padded
constexpr int kScratchBytes = kCounterBytes + 5 * kMaxChannels * (int)sizeof(float);

// The scratch of every call on this device.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels receive the device address obtained from it.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];   // per device, filled on the first call with that device current

// Prologue: clear the counters left by the previous call and fold the channel constants.
__global__ void static_prologue_kernel(cg_bn_params bn, const float* delta, float eps, int c_out,
                                       unsigned long long* counters, float* consts) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < CNT_SLOTS) counters[i] = 0ull;
  if (i < c_out) {
    const ChannelConsts k = fold_channel(bn, delta, eps, i);
    consts[i] = k.t;
    consts[c_out + i] = k.a1;
    consts[2 * c_out + i] = k.b1;
    consts[3 * c_out + i] = k.a2;
    consts[4 * c_out + i] = k.b2;
  }
}

// One warp per (pixel row, 32-channel block): base path, gate, conditional path where the gate
// fired, batch norm of the taken path, ReLU; the warp's ballot is the mask word (Section 3.1,
// Eq. 1-3, Section 4 of the paper).  Constants come from the scratch the prologue filled.
template <typename T>
__global__ void __launch_bounds__(256)
static_gated_conv_kernel(LayerDims L, const T* __restrict__ x, const T* __restrict__ w_base,
                         const T* __restrict__ w_cond, const float* __restrict__ consts,
                         const T* __restrict__ residual, T* __restrict__ y,
                         uint32_t* __restrict__ mask, unsigned long long* __restrict__ counters) {
  const float* c_t = consts;
  const float* c_a1 = consts + L.c_out;
  const float* c_b1 = consts + 2 * L.c_out;
  const float* c_a2 = consts + 3 * L.c_out;
  const float* c_b2 = consts + 4 * L.c_out;
  const int lane = threadIdx.x & 31;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  const long long warp0 = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long items = L.m * L.words;
  unsigned long long my_active = 0;
  for (long long it = warp0; it < items; it += warps) {
    const long long m = it / L.words;
    const int co = (int)(it - m * L.words) * 32 + lane;
    const int wo = (int)(m % L.wo);
    const int ho = (int)((m / L.wo) % L.ho);
    const int n = (int)(m / ((long long)L.wo * L.ho));
    bool fire = false;
    if (co < L.c_out) {
      const float p = conv_point<T>(L, x, w_base, n, ho, wo, co, 0, L.c_p);
      fire = (p >= c_t[co]);
      float v;
      if (fire) {
        const float r = conv_point<T>(L, x, w_cond, n, ho, wo, co, L.c_p, L.c_r);
        v = __fadd_rn(__fmul_rn(c_a2[co], __fadd_rn(p, r)), c_b2[co]);
      } else {
        v = __fadd_rn(__fmul_rn(c_a1[co], p), c_b1[co]);
      }
      if (residual) v = __fadd_rn(v, Elem<T>::ld(residual + m * L.c_out + co));
      if (L.relu) v = (v > 0.f) ? v : 0.f;
      st_out(y + m * L.c_out + co, v);
    }
    const unsigned word = __ballot_sync(0xffffffffu, fire);
    if (lane == 0) {
      if (mask) mask[it] = word;
      my_active += __popc(word);
    }
  }
  if (lane == 0 && my_active) atomicAdd(&counters[CNT_ACTIVE], my_active);
  if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd(&counters[CNT_CALLS], 1ull);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace
}  // namespace cg

extern "C" cg_status cg_conv_forward_static(const cg_conv_desc* d, const void* x, const void* w_base,
                                            const void* w_cond, const cg_bn_params* bn,
                                            const float* delta, const void* residual, void* y,
                                            uint32_t* mask_out, cg_stats* stats_out,
                                            void* cuda_stream) {
  using namespace cg;
  if (!d || !x || !w_base || !y || !bn || !delta) return CG_ERR_INVALID_ARG;
  if (d->n <= 0 || d->h <= 0 || d->w <= 0 || d->c_in <= 0 || d->c_out <= 0 || d->kh <= 0 ||
      d->kh != d->kw || d->stride <= 0 || d->pad < 0 || d->groups <= 0 || d->c_in % d->groups != 0 ||
      d->h + 2 * d->pad < d->kh || d->w + 2 * d->pad < d->kw || !(d->bn_eps >= 0.f))
    return CG_ERR_INVALID_ARG;
  if (d->in_dtype != d->out_dtype || (d->in_dtype != CG_F32 && d->in_dtype != CG_BF16))
    return CG_ERR_UNSUPPORTED;
  if (d->grouping || d->channel_tau > 0.f || bn->delta_high) return CG_ERR_UNSUPPORTED;
  if (d->c_out > kMaxChannels) return CG_ERR_WORKSPACE;   // would not fit the static scratch
  if (!bn->gamma || !bn->beta || !bn->mean_base || !bn->var_base || !bn->mean_full || !bn->var_full ||
      (bn->gate_mean == nullptr) != (bn->gate_var == nullptr))
    return CG_ERR_INVALID_ARG;
  if (!w_cond && d->c_in / d->groups != d->c_in) return CG_ERR_INVALID_ARG;
  if ((residual != nullptr) != (d->has_residual != 0)) return CG_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(w_base) || !aligned16(y) || (w_cond && !aligned16(w_cond)) ||
      (residual && !aligned16(residual)) || (reinterpret_cast<uintptr_t>(mask_out) & 3))
    return CG_ERR_ALIGNMENT;

  // address of the scratch array on the current device (first call on that device only)
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return CG_ERR_CUDA;
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return CG_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  unsigned char* scratch = static_cast<unsigned char*>(g_scratch_addr[dev]);
  unsigned long long* counters = reinterpret_cast<unsigned long long*>(scratch);
  float* consts = reinterpret_cast<float*>(scratch + kCounterBytes);

  LayerDims L;
  L.n = d->n; L.h = d->h; L.w = d->w; L.c_in = d->c_in; L.c_out = d->c_out;
  L.kh = d->kh; L.kw = d->kw; L.stride = d->stride; L.pad = d->pad;
  L.groups = d->groups; L.c_p = d->c_in / d->groups; L.c_r = d->c_in - L.c_p;
  L.ho = (d->h + 2 * d->pad - d->kh) / d->stride + 1;
  L.wo = (d->w + 2 * d->pad - d->kw) / d->stride + 1;
  L.m = (long long)d->n * L.ho * L.wo;
  L.words = (d->c_out + 31) / 32;
  L.eps = d->bn_eps; L.relu = d->relu ? 1 : 0; L.has_residual = d->has_residual ? 1 : 0; L.shift = 0; L.grouping = 0; L.channel_tau = 0.f;

  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int pro_threads = 256;
  const int pro_blocks = (max(d->c_out, (int)CNT_SLOTS) + pro_threads - 1) / pro_threads;
  static_prologue_kernel<<<pro_blocks, pro_threads, 0, stream>>>(*bn, delta, d->bn_eps, d->c_out,
                                                                 counters, consts);
  const long long items = L.m * L.words;
  long long blocks = (items + 7) / 8;
  if (blocks > 148ll * 64) blocks = 148ll * 64;
  if (d->in_dtype == CG_F32)
    static_gated_conv_kernel<float><<<(unsigned)blocks, 256, 0, stream>>>(
        L, (const float*)x, (const float*)w_base, (const float*)w_cond, consts,
        (const float*)residual, (float*)y, mask_out, counters);
  else
    static_gated_conv_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, stream>>>(
        L, (const __nv_bfloat16*)x, (const __nv_bfloat16*)w_base, (const __nv_bfloat16*)w_cond,
        consts, (const __nv_bfloat16*)residual, (__nv_bfloat16*)y, mask_out, counters);
  if (cudaGetLastError() != cudaSuccess) return CG_ERR_CUDA;

  if (stats_out) {
    unsigned long long c[CNT_SLOTS];
    if (cudaMemcpyAsync(c, counters, sizeof(c), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess)
      return CG_ERR_CUDA;
    const long long k2 = (long long)L.kh * L.kw;
    std::memset(stats_out, 0, sizeof(*stats_out));
    stats_out->calls = 1;
    stats_out->outputs = L.m * L.c_out;
    stats_out->active = (int64_t)c[CNT_ACTIVE];
    stats_out->dense_macs = stats_out->outputs * k2 * L.c_in;
    stats_out->gated_macs = k2 * ((long long)L.c_p * stats_out->outputs + (long long)L.c_r * stats_out->active);
    stats_out->executed_macs = stats_out->gated_macs;
    stats_out->channels = (int64_t)L.n * L.c_out;
  }
  return CG_OK;
}
