// Host side of the cgconv C ABI (include/cgconv.h): argument checks, kernel selection,
// counters.  No kernel lives here.
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"
#include "tc_conv.cuh"
#include "tc2_conv.cuh"
#include "tc3_conv.cuh"

struct cg_conv_s {
  cg_conv_desc desc;
  cg::LayerDims L;
  int use_tc;
  cg::TcPlan plan;
  int device;
  unsigned long long* counters;   // device, cg::CNT_SLOTS entries
  cg::TcMaps maps;                // tensor maps cached for the last set of pointers
  int use_tc2;                    // channel-major tensor-core kernel (tc2_conv.cu)
  cg::Tc2Plan plan2;
  cg::Tc2Maps maps2;
  int use_tc3;                    // tap-stacked tensor-core kernel (tc3_conv.cu)
  cg::Tc3Plan plan3;
  cg::Tc3Maps maps3;
};

namespace {

size_t elem_bytes(int dt) { return dt == CG_F32 ? 4 : (dt == CG_BF16 ? 2 : 1); }

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

cg_status check_desc(const cg_conv_desc* d) {
  if (!d) return CG_ERR_INVALID_ARG;
  if (d->n <= 0 || d->h <= 0 || d->w <= 0 || d->c_in <= 0 || d->c_out <= 0) return CG_ERR_INVALID_ARG;
  if (d->kh <= 0 || d->kw <= 0 || d->stride <= 0 || d->pad < 0) return CG_ERR_INVALID_ARG;
  if (d->kh != d->kw) return CG_ERR_INVALID_ARG;
  if (d->groups <= 0 || d->c_in % d->groups != 0) return CG_ERR_INVALID_ARG;
  if ((d->h + 2 * d->pad - d->kh) < 0 || (d->w + 2 * d->pad - d->kw) < 0) return CG_ERR_INVALID_ARG;
  if (d->in_dtype != CG_F32 && d->in_dtype != CG_BF16 && d->in_dtype != CG_I8) return CG_ERR_INVALID_ARG;
  if (d->out_dtype != d->in_dtype) return CG_ERR_INVALID_ARG;
  if (d->in_dtype == CG_I8 && (d->requant_shift < 1 || d->requant_shift > 31)) return CG_ERR_INVALID_ARG;
  if (d->in_dtype == CG_I8 && d->has_residual) return CG_ERR_INVALID_ARG;
  if (!(d->bn_eps >= 0.f)) return CG_ERR_INVALID_ARG;
  if (d->algo < CG_ALGO_AUTO || d->algo > CG_ALGO_TENSOR_STACKED) return CG_ERR_INVALID_ARG;
  if (d->cond_mode < CG_COND_AUTO || d->cond_mode > CG_COND_COMPACT) return CG_ERR_INVALID_ARG;
  if (d->grouping != 0 && d->grouping != 1) return CG_ERR_INVALID_ARG;
  if (d->grouping && d->c_out % d->groups != 0) return CG_ERR_INVALID_ARG;
  if (d->grouping && d->in_dtype == CG_I8) return CG_ERR_INVALID_ARG;   // not defined for I8 layers
  if (!(d->channel_tau >= 0.f)) return CG_ERR_INVALID_ARG;               // negative or NaN
  if (d->channel_tau > 0.f && d->in_dtype == CG_I8) return CG_ERR_INVALID_ARG;
  return CG_OK;
}

cg::LayerDims make_dims(const cg_conv_desc& d) {
  cg::LayerDims L;
  L.n = d.n; L.h = d.h; L.w = d.w; L.c_in = d.c_in; L.c_out = d.c_out;
  L.kh = d.kh; L.kw = d.kw; L.stride = d.stride; L.pad = d.pad;
  L.groups = d.groups; L.c_p = d.c_in / d.groups; L.c_r = d.c_in - L.c_p;
  L.ho = (d.h + 2 * d.pad - d.kh) / d.stride + 1;
  L.wo = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
  L.m = (long long)d.n * L.ho * L.wo;
  L.words = (d.c_out + 31) / 32;
  L.eps = d.bn_eps; L.relu = d.relu ? 1 : 0; L.has_residual = d.has_residual ? 1 : 0;
  L.shift = d.requant_shift;
  L.grouping = d.grouping;
  L.channel_tau = d.channel_tau;
  return L;
}

cg_status check_bn(const cg_conv_s* h, const cg_bn_params* bn, const float* delta) {
  if (!bn) return CG_ERR_INVALID_ARG;
  if (h->desc.in_dtype == CG_I8) {
    if (!bn->q_gate_thr || !bn->q_mul_base || !bn->q_mul_full || !bn->q_off_base || !bn->q_off_full)
      return CG_ERR_INVALID_ARG;
    if (bn->delta_high) return CG_ERR_INVALID_ARG;      // the two-sided gate is defined for floating-point layers
  } else {
    if (!bn->gamma || !bn->beta || !bn->mean_base || !bn->var_base || !bn->mean_full || !bn->var_full)
      return CG_ERR_INVALID_ARG;
    if ((bn->gate_mean == nullptr) != (bn->gate_var == nullptr)) return CG_ERR_INVALID_ARG;
    if (!delta) return CG_ERR_INVALID_ARG;
  }
  return CG_OK;
}

}  // namespace

extern "C" {

const char* cg_status_string(cg_status s) {
  switch (s) {
    case CG_OK: return "ok";
    case CG_ERR_INVALID_ARG: return "invalid argument";
    case CG_ERR_UNSUPPORTED: return "layer not supported by the requested kernels";
    case CG_ERR_ALIGNMENT: return "tensor pointer not sufficiently aligned";
    case CG_ERR_WORKSPACE: return "workspace missing or too small";
    case CG_ERR_CUDA: return "CUDA call failed";
    case CG_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired";
    case CG_ERR_DEVICE_BOUNDS: return "a kernel-side range check failed";
  }
  return "unknown status";
}

cg_status cg_conv_create(cg_conv_t* out, const cg_conv_desc* desc) {
  if (!out) return CG_ERR_INVALID_ARG;
  const cg_status st = check_desc(desc);
  if (st != CG_OK) return st;
  cg_conv_s* h = new (std::nothrow) cg_conv_s();
  if (!h) return CG_ERR_INVALID_ARG;
  h->desc = *desc;
  h->L = make_dims(*desc);
  h->counters = nullptr;
  std::memset(&h->maps, 0, sizeof(h->maps));
  std::memset(&h->maps2, 0, sizeof(h->maps2));
  std::memset(&h->maps3, 0, sizeof(h->maps3));
  // (which kernels apply is decided before the device is needed, so that an ineligible layer is
  // reported as such on any machine)
  const bool have_device = cudaGetDevice(&h->device) == cudaSuccess;
  int sms = 0;
  if (!have_device || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess || sms <= 0) sms = 148;
  // the channel-wise gate needs every partial sum of an image before any conditional path: it
  // runs as two passes of the pixel-major kernel (chan_gate.cu), or on the direct kernels
  const bool chan = desc->channel_tau > 0.f;
  const bool want_tc = desc->algo != CG_ALGO_DIRECT;
  // Two tensor-core kernels.  Measured on B200 (batch 64-256 ResNet-18 shapes), the channel-major
  // kernel is the faster one for 128 output channels, and for 256 channels on 8x8 images (where the
  // pixel-major kernel's whole-image tiles are half padding) or with 20,000 and more pixels (enough
  // pixel tiles to fill every SM with both channel tiles); elsewhere the pixel-major kernel wins.
  // Each also takes the layers only it can run.
  const bool prefer2 = h->L.c_out == 128 ||
                       (h->L.c_out == 256 && (h->L.ho * h->L.wo <= 64 || h->L.m >= 20000));
  // A third kernel takes the 64 -> 64 channel layers it can run (measured faster than both others).
  const bool only3 = desc->algo == CG_ALGO_TENSOR_STACKED;
  const bool allow1 = desc->algo != CG_ALGO_TENSOR_CHANNELS && !only3;
  const bool allow2 = desc->algo != CG_ALGO_TENSOR_ROWS && !chan && !only3;
  const bool allow3 = desc->algo == CG_ALGO_AUTO || desc->algo == CG_ALGO_TENSOR || only3;
  const int cond_mode = (chan && desc->cond_mode == CG_COND_COMPACT) ? CG_COND_SKIP_TILES : desc->cond_mode;
  bool ok1 = false, ok2 = false;
  h->use_tc3 = want_tc && allow3 && cg::tc3_plan(h->L, desc->in_dtype, cond_mode, sms, &h->plan3);
  // (image widths that do not divide 32 make the kernel's warps exchange edge values: measured slower
  // than the pixel-major kernel, 47 against 38 us on 64 images of 56x56, so only an explicit request
  // runs them there)
  if (h->use_tc3 && h->plan3.xch && !only3) h->use_tc3 = 0;
  if (!h->use_tc3 && want_tc && allow2 && (prefer2 || !allow1)) ok2 = cg::tc2_plan(h->L, desc->in_dtype, cond_mode, sms, &h->plan2);
  if (want_tc && allow1 && !ok2 && !h->use_tc3) ok1 = cg::tc_plan(h->L, desc->in_dtype, cond_mode, &h->plan);
  if (want_tc && allow2 && !ok1 && !ok2 && !h->use_tc3) ok2 = cg::tc2_plan(h->L, desc->in_dtype, cond_mode, sms, &h->plan2);
  h->use_tc2 = ok2;
  const bool tc_ok = ok1;
  const bool must_tc = desc->algo >= CG_ALGO_TENSOR;
  if (must_tc && !tc_ok && !h->use_tc2 && !h->use_tc3) { delete h; return CG_ERR_UNSUPPORTED; }
  if (!have_device) { delete h; return CG_ERR_CUDA; }
  h->use_tc = tc_ok || h->use_tc2 || h->use_tc3;
  if (h->use_tc && !cg::tc_device_ok(h->device)) {
    if (must_tc) { delete h; return CG_ERR_UNSUPPORTED; }
    h->use_tc = 0; h->use_tc2 = 0; h->use_tc3 = 0;
  }
  if (cudaMalloc(&h->counters, cg::CNT_SLOTS * sizeof(unsigned long long)) != cudaSuccess) {
    delete h; return CG_ERR_CUDA;
  }
  if (cudaMemset(h->counters, 0, cg::CNT_SLOTS * sizeof(unsigned long long)) != cudaSuccess) {
    cudaFree(h->counters); delete h; return CG_ERR_CUDA;
  }
  *out = h;
  return CG_OK;
}

void cg_conv_destroy(cg_conv_t h) {
  if (!h) return;
  if (h->counters) cudaFree(h->counters);
  delete h;
}

size_t cg_conv_workspace_bytes(cg_conv_t h) {
  if (!h) return 0;
  if (h->L.channel_tau > 0.f && h->use_tc) return cg::tc_channel_gate_workspace_bytes(h->L, h->plan);
  if (h->L.channel_tau > 0.f) return cg::channel_gate_workspace_bytes(h->L);
  if (h->use_tc2) return cg::tc2_workspace_bytes(h->L, h->plan2);
  if (h->use_tc3) return 0;
  return h->use_tc ? cg::tc_workspace_bytes(h->L, h->plan) : 0;
}

int cg_conv_launches_per_forward(cg_conv_t h) {
  if (!h) return 0;
  if (h->L.channel_tau > 0.f) return h->use_tc ? 4 + 2 * (h->plan.pad8 ? 1 : 0) : 2;
  if (h->use_tc2) return h->plan2.pad8 ? 2 : 1;
  if (h->use_tc3) return 1;
  return (h->use_tc && (h->plan.cond_mode == CG_COND_COMPACT || h->plan.pad8)) ? 2 : 1;
}

int cg_conv_uses_tensor_cores(cg_conv_t h) { return h ? h->use_tc : 0; }

int cg_conv_plan_string(cg_conv_t h, char* buf, size_t len) {
  if (!h || !buf || len == 0) return -1;
  if (h->use_tc2) {
    const cg::Tc2Plan& P = h->plan2;
    return std::snprintf(buf, len,
                         "channel-major tcgen05: %d channel tile(s) x %d pixel tiles of %d sub-tile(s) x %d stacked rows "
                         "(%d pixels, MMA N=%d), %d K stages (%d base), weight ring %d, lead %d, grid %d",
                         P.tiles_c, P.jobs_m, P.nsub, P.r, P.np, P.nmma, P.ns, P.nb, P.ring, P.lead, P.grid);
  }
  if (h->use_tc3) {
    const cg::Tc3Plan& P = h->plan3;
    return std::snprintf(buf, len,
                         "tap-stacked tcgen05: %d jobs of %d image rows (128 pixels x 192 stacked columns), %d base K step(s) "
                         "of 4, resident weights, grid %d",
                         P.jobs, P.rows, P.kp, P.grid);
  }
  if (h->use_tc) {
    const cg::TcPlan& P = h->plan;
    return std::snprintf(buf, len,
                         "pixel-major tcgen05: %d row tiles x %d column tiles of %d, %s weights, %d patch buffers, %d issuer(s)",
                         P.tiles_m, P.tiles_n, P.nt, P.resident ? "resident" : "streamed", P.na, P.issuers);
  }
  return std::snprintf(buf, len, "direct CUDA-core kernels");
}

int cg_conv_kernel_id(cg_conv_t h) {
  if (!h) return -1;
  if (h->use_tc3) return CG_KERNEL_TENSOR_TAP_STACKED;
  return h->use_tc2 ? CG_KERNEL_TENSOR_CHANNEL_MAJOR : (h->use_tc ? CG_KERNEL_TENSOR_PIXEL_MAJOR : CG_KERNEL_DIRECT);
}

cg_status cg_conv_forward(cg_conv_t h, const void* x, const void* w_base, const void* w_cond,
                          const cg_bn_params* bn, const float* delta, const void* residual,
                          void* y, uint32_t* mask_out, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
  if (!h || !x || !w_base || !y) return CG_ERR_INVALID_ARG;
  if (!w_cond && h->L.c_r > 0) return CG_ERR_INVALID_ARG;
  cg_status st = check_bn(h, bn, delta);
  if (st != CG_OK) return st;
  if ((residual != nullptr) != (h->desc.has_residual != 0)) return CG_ERR_INVALID_ARG;
  if (!aligned(x, 16) || !aligned(w_base, 16) || (w_cond && !aligned(w_cond, 16)) ||
      !aligned(y, 16) || (residual && !aligned(residual, 16)) || (mask_out && !aligned(mask_out, 4)))
    return CG_ERR_ALIGNMENT;
  const size_t need = cg_conv_workspace_bytes(h);
  if (need > 0 && (!workspace || workspace_bytes < need)) return CG_ERR_WORKSPACE;
  // the kernels that use the workspace access it in 16-byte pieces and clear its first 256 bytes
  if (need > 0 && !aligned(workspace, 256)) return CG_ERR_ALIGNMENT;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return CG_ERR_CUDA;
  if (cur != h->device) return CG_ERR_INVALID_ARG;         // a handle belongs to the device it was created on
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  int err;
  if (h->use_tc && h->L.channel_tau > 0.f) {
    err = cg::launch_tc_channel_gate(h->L, h->plan, h->desc.in_dtype, &h->maps, x, w_base, w_cond, *bn, delta,
                                     residual, y, mask_out, workspace, h->counters, stream);
  } else if (h->use_tc3) {
    err = cg::launch_tc3(h->L, h->plan3, &h->maps3, x, w_base, w_cond, *bn, delta, residual, y, mask_out,
                         h->counters, stream);
  } else if (h->use_tc2) {
    err = cg::launch_tc2(h->L, h->plan2, &h->maps2, x, w_base, w_cond, *bn, delta, residual, y,
                         mask_out, workspace, h->counters, stream);
  } else if (h->use_tc) {
    err = cg::launch_tc(h->L, h->plan, h->desc.in_dtype, &h->maps, x, w_base, w_cond, *bn, delta,
                        residual, y, mask_out, workspace, h->counters, stream);
  } else if (h->L.channel_tau > 0.f) {
    err = cg::launch_direct_channel_gate(h->L, h->desc.in_dtype, x, w_base, w_cond, *bn, delta,
                                         residual, y, mask_out, workspace, h->counters, stream);
  } else {
    err = cg::launch_direct(h->L, h->desc.in_dtype, x, w_base, w_cond, *bn, delta, residual, y,
                            mask_out, nullptr, 0, h->counters, stream);
  }
  if (err != 0) return CG_ERR_CUDA;
  return CG_OK;
}

size_t cg_conv_host_staging_bytes(cg_conv_t h) {
  if (!h) return 0;
  const size_t eb = elem_bytes(h->desc.in_dtype), ob = elem_bytes(h->desc.out_dtype);
  size_t total = align_up((size_t)h->L.n * h->L.h * h->L.w * h->L.c_in * eb, 256);
  total += align_up((size_t)h->L.m * h->L.c_out * ob, 256);                     // y
  total += align_up((size_t)h->L.m * h->L.words * 4, 256);                      // mask
  if (h->desc.has_residual) total += align_up((size_t)h->L.m * h->L.c_out * ob, 256);
  total += align_up(cg_conv_workspace_bytes(h), 256);
  return total;
}

cg_status cg_conv_forward_host(cg_conv_t h, const void* x_host, const void* w_base,
                               const void* w_cond, const cg_bn_params* bn, const float* delta,
                               const void* residual_host, void* y_host, uint32_t* mask_host,
                               void* staging, size_t staging_bytes, void* cuda_stream) {
  if (!h || !x_host || !y_host || !staging) return CG_ERR_INVALID_ARG;
  if (staging_bytes < cg_conv_host_staging_bytes(h)) return CG_ERR_WORKSPACE;
  if (!aligned(staging, 256)) return CG_ERR_ALIGNMENT;
  if ((residual_host != nullptr) != (h->desc.has_residual != 0)) return CG_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t eb = elem_bytes(h->desc.in_dtype), ob = elem_bytes(h->desc.out_dtype);
  const size_t x_bytes = (size_t)h->L.n * h->L.h * h->L.w * h->L.c_in * eb;
  const size_t y_bytes = (size_t)h->L.m * h->L.c_out * ob;
  const size_t m_bytes = (size_t)h->L.m * h->L.words * 4;
  char* p = static_cast<char*>(staging);
  void* x_dev = p; p += align_up(x_bytes, 256);
  void* y_dev = p; p += align_up(y_bytes, 256);
  uint32_t* m_dev = reinterpret_cast<uint32_t*>(p); p += align_up(m_bytes, 256);
  void* r_dev = nullptr;
  if (h->desc.has_residual) { r_dev = p; p += align_up(y_bytes, 256); }
  void* ws = p;
  if (cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return CG_ERR_CUDA;
  if (r_dev && cudaMemcpyAsync(r_dev, residual_host, y_bytes, cudaMemcpyHostToDevice, stream) !=
                   cudaSuccess)
    return CG_ERR_CUDA;
  const cg_status st = cg_conv_forward(h, x_dev, w_base, w_cond, bn, delta, r_dev, y_dev,
                                       mask_host ? m_dev : nullptr, ws,
                                       cg_conv_workspace_bytes(h), cuda_stream);
  if (st != CG_OK) return st;
  if (cudaMemcpyAsync(y_host, y_dev, y_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return CG_ERR_CUDA;
  if (mask_host &&
      cudaMemcpyAsync(mask_host, m_dev, m_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return CG_ERR_CUDA;
  return CG_OK;
}

cg_status cg_conv_partial_sums(cg_conv_t h, const void* x, const void* w_base, void* p_out,
                               void* cuda_stream) {
  if (!h || !x || !w_base || !p_out) return CG_ERR_INVALID_ARG;
  if (!aligned(x, 16) || !aligned(w_base, 16) || !aligned(p_out, 4)) return CG_ERR_ALIGNMENT;
  cg_bn_params none;
  std::memset(&none, 0, sizeof(none));
  const int err = cg::launch_direct(h->L, h->desc.in_dtype, x, w_base, nullptr, none, nullptr,
                                    nullptr, nullptr, nullptr, p_out, 1, h->counters,
                                    reinterpret_cast<cudaStream_t>(cuda_stream));
  return err == 0 ? CG_OK : CG_ERR_CUDA;
}

cg_status cg_conv_stats(cg_conv_t h, cg_stats* out, void* cuda_stream) {
  if (!h || !out) return CG_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  unsigned long long c[cg::CNT_SLOTS];
  if (cudaMemcpyAsync(c, h->counters, sizeof(c), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
    return CG_ERR_CUDA;
  if (cudaMemsetAsync(h->counters, 0, sizeof(c), stream) != cudaSuccess) return CG_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return CG_ERR_CUDA;
  const cg::LayerDims& L = h->L;
  const long long k2 = (long long)L.kh * L.kw;
  std::memset(out, 0, sizeof(*out));
  out->calls = (int64_t)c[cg::CNT_CALLS];
  out->outputs = out->calls * L.m * L.c_out;
  out->active = (int64_t)c[cg::CNT_ACTIVE];
  out->dense_macs = out->outputs * k2 * L.c_in;
  out->gated_macs = k2 * ((long long)L.c_p * out->outputs + (long long)L.c_r * out->active);
  // the tensor-core kernels count every MMA they issue (base path included, at tile
  // granularity); the direct kernels execute exactly the method's count
  out->executed_macs = h->use_tc ? (int64_t)c[cg::CNT_EXEC_MACS] : out->gated_macs;
  out->tiles_total = (int64_t)c[cg::CNT_TILES_TOTAL];
  out->tiles_skipped = (int64_t)c[cg::CNT_TILES_SKIPPED];
  out->rows_total = (int64_t)c[cg::CNT_ROWS_TOTAL];
  out->rows_active = (int64_t)c[cg::CNT_ROWS_ACTIVE];
  out->device_status = (int32_t)c[cg::CNT_STATUS];
  out->device_site = (int32_t)c[cg::CNT_SITE];
  out->channels = out->calls * L.n * L.c_out;
  out->channels_skipped = (int64_t)c[cg::CNT_CH_SKIPPED];
  return out->device_status ? (cg_status)out->device_status : CG_OK;
}

}  // extern "C"
