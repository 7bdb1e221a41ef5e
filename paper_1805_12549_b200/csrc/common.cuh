// Shared declarations of the cgconv CUDA library (host API <-> kernel launchers).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cgconv.h"

namespace cg {

// Layer geometry handed to every kernel by value.
struct LayerDims {
  int n, h, w, c_in, c_out;
  int kh, kw, stride, pad;
  int groups, c_p, c_r;   // c_p = c_in / G base channels, c_r = c_in - c_p
  int ho, wo;             // output extents
  long long m;            // n * ho * wo pixel rows
  int words;              // ceil(c_out / 32) mask words per pixel row
  float eps;
  int relu, has_residual, shift;
  int grouping;           // 1: output group i uses input group i as x_p (Section 3.3)
  float channel_tau;      // > 0: channel-wise gate (Eq. 4)
};

// Device counter block owned by a handle: 16 x u64.
enum CounterSlot {
  CNT_ACTIVE = 0,
  CNT_EXEC_MACS = 1,
  CNT_TILES_TOTAL = 2,
  CNT_TILES_SKIPPED = 3,
  CNT_ROWS_TOTAL = 4,
  CNT_ROWS_ACTIVE = 5,
  CNT_STATUS = 6,   // first non-zero cg_status reported by a kernel
  CNT_SITE = 7,     // id of the wait/check that reported it
  CNT_CALLS = 8,    // forward passes executed (counted on the device: graph replays count)
  CNT_CH_SKIPPED = 9,   // (image, output channel) pairs switched off by the channel-wise gate
  CNT_SLOTS = 16
};

// Batch-norm / gate constants of one output channel, in fp32 with separately rounded
// operations:  t = Delta*sqrt(var_g+eps) + mean_g  (Eq. 3, merged gate);
// a = gamma/sqrt(var+eps), b = beta - a*mean  (a batch norm at inference is a scale and shift).
struct ChannelConsts {
  float t, a1, b1, a2, b2;
  float t2;   // upper threshold of the two-sided gate (Section 3.2); +inf for the one-sided gate
};

__device__ __forceinline__ ChannelConsts fold_channel(const cg_bn_params& bn, const float* delta,
                                                      float eps, int c) {
  ChannelConsts k;
  const float* gm = bn.gate_mean ? bn.gate_mean : bn.mean_base;
  const float* gv = bn.gate_var ? bn.gate_var : bn.var_base;
  const float sg = __fsqrt_rn(__fadd_rn(gv[c], eps));
  k.t = __fadd_rn(__fmul_rn(delta[c], sg), gm[c]);
  k.t2 = bn.delta_high ? __fadd_rn(__fmul_rn(bn.delta_high[c], sg), gm[c]) : __int_as_float(0x7f800000);
  const float g = bn.gamma[c], be = bn.beta[c];
  k.a1 = __fdiv_rn(g, __fsqrt_rn(__fadd_rn(bn.var_base[c], eps)));
  k.b1 = __fsub_rn(be, __fmul_rn(k.a1, bn.mean_base[c]));
  k.a2 = __fdiv_rn(g, __fsqrt_rn(__fadd_rn(bn.var_full[c], eps)));
  k.b2 = __fsub_rn(be, __fmul_rn(k.a2, bn.mean_full[c]));
  return k;
}

// ---- launchers (each returns a cudaError_t-compatible int; 0 = success) -----------------
int launch_direct(const LayerDims& L, int in_dtype, const void* x, const void* w_base,
                  const void* w_cond, const cg_bn_params& bn, const float* delta,
                  const void* residual, void* y, uint32_t* mask, void* p_out, int base_only,
                  unsigned long long* counters, cudaStream_t stream);
// Layer with the channel-wise gate (Eq. 4), floating point only: partial sums and per-(image,
// channel) counts, then the conditional path under both gates.  workspace as sized by
// channel_gate_workspace_bytes.
size_t channel_gate_workspace_bytes(const LayerDims& L);
int launch_direct_channel_gate(const LayerDims& L, int in_dtype, const void* x, const void* w_base,
                               const void* w_cond, const cg_bn_params& bn, const float* delta,
                               const void* residual, void* y, uint32_t* mask, void* workspace,
                               unsigned long long* counters, cudaStream_t stream);

}  // namespace cg
