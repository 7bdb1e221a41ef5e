/* cgconv -- channel-gated convolution layer for NVIDIA B200 (sm_100a).
 *
 * C ABI of the inference forward pass of the channel-gating block defined in
 * "Channel Gating Neural Networks" (arXiv 1805.12549):
 *
 *   Section 3.1   the input channels are split statically, x = [x_p, x_r]; the
 *                 base path W_p*x_p is computed for every output activation;
 *   Eq. 2, Eq. 3  the gate d = theta(P - Delta*sqrt(Var) - E) on the partial sum
 *                 P, one threshold per output channel, a tie fires;
 *   Eq. 1         the conditional path W_r*x_r is needed only where d = 1, and
 *                 y = f(P) where d = 0, y = f(P + R) where d = 1;
 *   Section 4     the two results go through two batch norms (BN1 for P, BN2
 *                 for P+R) that share gamma and beta; at inference each is a
 *                 per-channel scale and shift; f is ReLU.
 *
 * Tensors are NHWC.  GEMM view: M = n*h'*w' pixel rows, c_out columns.
 * Every tensor argument of cg_conv_forward is a DEVICE pointer owned by the
 * caller; the library never allocates in cg_conv_forward.  Calls return a
 * status code; nothing throws, aborts or traps.
 */
#ifndef CGCONV_H_
#define CGCONV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cg_conv_s* cg_conv_t; /* opaque handle, owned by the library */

typedef enum {
  CG_OK = 0,
  CG_ERR_INVALID_ARG = 1,    /* NULL pointer, non-positive extent, inconsistent description */
  CG_ERR_UNSUPPORTED = 2,    /* valid layer that this build has no kernel for                */
  CG_ERR_ALIGNMENT = 3,      /* a tensor pointer is not 16-byte aligned                      */
  CG_ERR_WORKSPACE = 4,      /* workspace missing or smaller than cg_conv_workspace_bytes    */
  CG_ERR_CUDA = 5,           /* a CUDA runtime/driver call failed (no device, launch error)  */
  CG_ERR_DEVICE_TIMEOUT = 6, /* a bounded wait inside a kernel gave up (see cg_stats)        */
  CG_ERR_DEVICE_BOUNDS = 7   /* a kernel-side range check failed (see cg_stats)              */
} cg_status;

typedef enum { CG_F32 = 0, CG_BF16 = 1, CG_I8 = 2 } cg_dtype;

/* Which kernels run the layer. */
typedef enum {
  CG_ALGO_AUTO = 0,   /* tensor-core path when the layer qualifies, else the direct path */
  CG_ALGO_DIRECT = 1, /* CUDA-core direct convolution: any shape, sums in the order (r,s,c_in) */
  CG_ALGO_TENSOR = 2, /* tcgen05 implicit GEMM; CG_ERR_UNSUPPORTED at create if not eligible */
  CG_ALGO_TENSOR_ROWS = 3,     /* the pixel-major tcgen05 kernel only (pixels on the MMA's M side) */
  CG_ALGO_TENSOR_CHANNELS = 4, /* the channel-major tcgen05 kernel only (output channels on the M side) */
  CG_ALGO_TENSOR_STACKED = 5   /* the tap-stacked tcgen05 kernel only (64 -> 64 channel layers: the three
                                  taps of a filter row share one MMA).
                                  AUTO and TENSOR pick between the three by layer shape. */
} cg_algo;

/* How the tensor-core path treats the conditional path (Eq. 1, second case). */
typedef enum {
  CG_COND_AUTO = 0,
  CG_COND_DENSE = 1,     /* compute R for every row of every tile (gate density 1.0 behaviour)  */
  CG_COND_SKIP_TILES = 2,/* skip tiles (and column blocks) in which no gate fired               */
  CG_COND_COMPACT = 3    /* additionally gather only the pixel rows in which a gate fired       */
} cg_cond_mode;

/* Layer description, fixed at create time. */
typedef struct {
  int32_t n, h, w, c_in, c_out; /* input extents [n,h,w,c_in]; output channels                */
  int32_t kh, kw, stride, pad;  /* square kernels only (kh == kw); zero padding; floor output
                                   size h' = (h + 2*pad - kh)/stride + 1                       */
  int32_t groups;               /* G = 1/eta (Section 3.1): the base path reads input channels
                                   [0, c_in/G), the conditional path the rest.  G = 1: ungated */
  int32_t in_dtype;             /* cg_dtype of x, w_base, w_cond                               */
  int32_t out_dtype;            /* cg_dtype of y, equal to in_dtype (a BF16 layer with I8
                                   output is not built: CG_ERR_INVALID_ARG)                    */
  float bn_eps;                 /* added inside sqrt(var + eps) of BN1, BN2 and the gate       */
  int32_t relu;                 /* 1: f = ReLU (the paper's choice); 0: identity               */
  int32_t has_residual;         /* 1: `residual` [M,c_out] (out_dtype) is added after the batch
                                   norm and before f.  Not part of the paper's block.          */
  int32_t requant_shift;        /* I8 only: S in [1,31]                                        */
  int32_t algo;                 /* cg_algo                                                     */
  int32_t cond_mode;            /* cg_cond_mode (tensor-core path only)                        */
  int32_t grouping;             /* 0: every output channel takes input channels [0,c_in/G) as
                                   x_p (Fig. 5(a)).  1: channel grouping (Section 3.3, Fig. 5(b)):
                                   output group i = channels [i*c_out/G,(i+1)*c_out/G) takes input
                                   group i as x_p and the other groups, in ascending order, as
                                   x_r; needs c_out % G == 0.  Tensor-core kernels where an
                                   input group is whole 64-channel chunks and an output group a
                                   multiple of 64 (128) channels; direct kernels otherwise.     */
  float channel_tau;            /* tau_c of the channel-wise gate (Eq. 4).  0: off.  > 0: per
                                   image, an output channel whose gate fires at fewer than
                                   tau_c * h' * w' positions loses its conditional path (all its
                                   activations take Eq. 1's first case, its mask bits are 0);
                                   a count equal to tau_c*h'*w' keeps the channel (theta(0) = 1);
                                   the comparison is (float)count >= tau_c * (float)(h'*w').
                                   Floating-point layers.  BF16 layers the pixel-major tensor-core
                                   kernel can run take two passes of it (base path and gate; the
                                   whole layer with per-image thresholds) with two small kernels
                                   in between; other layers run on the direct kernels (a memset of
                                   the counts and two launches).  Needs the workspace
                                   cg_conv_workspace_bytes reports.                            */
} cg_conv_desc;

/* Per-output-channel parameters: DEVICE pointers to c_out entries, caller-owned.
 * Floating-point layers use the float members; I8 layers use the q_* members. */
typedef struct {
  const float* gamma;     /* shared by BN1 and BN2 (Section 4, footnote)                       */
  const float* beta;
  const float* mean_base; /* BN1: running statistics of P                                      */
  const float* var_base;
  const float* mean_full; /* BN2: running statistics of P + R                                  */
  const float* var_full;
  const float* gate_mean; /* E[x], Var(x) of Eq. 3; both NULL => BN1's statistics              */
  const float* gate_var;
  /* I8 layers (a convention of this library; the paper does not give its quantisation):
   *   d = (P >= q_gate_thr[c]); acc = d ? P+R : P (int32);
   *   z = (int64)acc * q_mul_sel[c] + q_off_sel[c], sel = full if d else base;
   *   q = (z + 2^(S-1)) >> S (arithmetic shift);  y = clamp(q, relu ? 0 : -128, 127).        */
  const int32_t* q_gate_thr;
  const int32_t* q_mul_base;
  const int32_t* q_mul_full;
  const int64_t* q_off_base;
  const int64_t* q_off_full;
  /* Two-sided gate of Section 3.2, s = theta(Delta_h - x) o theta(x - Delta_l), for networks whose
   * activation saturates on both sides: upper thresholds Delta_h[c] in the same normalised units
   * as `delta` (which is then Delta_l); a gate fires iff Delta_l <= x^ <= Delta_h, ties included.
   * NULL: the one-sided gate theta(x - Delta).  Floating-point layers only. */
  const float* delta_high;
} cg_bn_params;

/* Counters accumulated by cg_conv_forward since the last cg_conv_stats. */
typedef struct {
  int64_t calls;         /* forward calls counted                                              */
  int64_t outputs;       /* calls * M * c_out                                                  */
  int64_t active;        /* activations whose gate fired (d = 1)                               */
  int64_t dense_macs;    /* multiplications of the ungated layer: outputs * k^2 * c_in         */
  int64_t gated_macs;    /* the method's count (Section 4): k^2*(c_p*outputs + c_r*active)     */
  int64_t executed_macs; /* multiplications the kernels really issued, at tile/row granularity */
  int64_t tiles_total;   /* conditional-path tiles (row block x column block) considered       */
  int64_t tiles_skipped; /* ... of which skipped because no gate fired in them                 */
  int64_t rows_total;    /* pixel rows x column blocks considered                              */
  int64_t rows_active;   /* ... of which contained at least one firing gate                    */
  int32_t device_status; /* CG_OK, CG_ERR_DEVICE_TIMEOUT or CG_ERR_DEVICE_BOUNDS               */
  int32_t device_site;   /* which wait/check reported it (kernel-internal id), 0 if none       */
  int64_t channels;         /* calls * n * c_out: output channels, one per image (Eq. 4)       */
  int64_t channels_skipped; /* ... of which the channel-wise gate switched off (their
                               conditional weights need not be fetched); 0 when channel_tau = 0 */
} cg_stats;

/* Section 3.1: fixes the layer and picks kernels.  Host work only, plus one small device
 * allocation for the counters (freed by cg_conv_destroy).  `*out` is set on CG_OK only.
 * Errors: CG_ERR_INVALID_ARG (NULL, extents <= 0, c_in % groups != 0, kh != kw, dtype pair not
 * listed above, shift out of range), CG_ERR_CUDA, and CG_ERR_UNSUPPORTED when a tensor-core
 * algo is asked for a layer outside the kernels' limits.  Those are: BF16 or I8; the channel-wise
 * gate on the pixel-major kernel only; channel grouping only for BF16 with c_in/G a multiple of 64 and c_out/G a multiple of 64
 * (pixel-major) or 128 (channel-major); odd square filter with pad = (k-1)/2; c_in a multiple of 64
 * (BF16), a multiple of 128 or equal to 64 (I8);
 *   pixel-major kernel:   stride 1, or stride 2 for 3x3 filters on even extents; c_out a multiple
 *                         of 64; c_in/G equal to 8, 16 or 32 (BF16; 32 or 64 for I8, at most 32 when
 *                         c_in = 64) or a multiple of 64 (128); output width at most 128;
 *   channel-major kernel: BF16, stride 1, c_out a multiple of 32, c_in/G equal to 8, 16, 32 or a
 *                         multiple of 64, no row compaction (CG_COND_COMPACT);
 *   tap-stacked kernel:   BF16, 3x3, stride 1, pad 1, c_in = c_out = 64, c_in/G a multiple of 16, image
 *                         width at most 128, no channel grouping, no channel-wise gate, no row compaction
 *                         (AUTO and TENSOR choose it when the width divides 32).
 * AUTO falls back to the direct kernels outside these limits.
 * A handle is not thread-safe: calls on one handle must not overlap in time on the host
 * (different handles are independent).  Forward calls of one handle may be queued on different
 * streams only if the streams are ordered so that they do not run concurrently: the counters and
 * the workspace are per handle. */
cg_status cg_conv_create(cg_conv_t* out, const cg_conv_desc* desc);

/* Bytes of device scratch cg_conv_forward needs (may be 0): the partial sums and per-channel
 * counts of the channel-wise gate (Eq. 4), the compacted row lists of CG_COND_COMPACT (Eq. 1: the
 * rows where d = 1), or weights repacked with whole K steps (c_in/G = 8; I8 layers with c_in = 64).  Contents need not persist between
 * calls; two forwards that overlap in time must not share one workspace.  The pointer given to
 * cg_conv_forward must be 256-byte aligned (CG_ERR_ALIGNMENT otherwise). */
size_t cg_conv_workspace_bytes(cg_conv_t h);

/* Eq. 1-3 and the two batch norms of Section 4 for one batch.
 *   x         [n,h,w,c_in] in_dtype
 *   w_base    [c_out,kh,kw,c_in/G] in_dtype            (W_p)
 *   w_cond    [c_out,kh,kw,c_in-c_in/G] in_dtype       (W_r; ignored when G = 1, may be NULL)
 *   bn        host struct of device pointers (read during the call, not kept)
 *   delta     [c_out] float, Delta of Eq. 3 in normalised units, +-inf allowed (all shut /
 *             all open); ignored (may be NULL) for I8, which uses bn->q_gate_thr
 *   residual  [M,c_out] out_dtype or NULL (must be NULL unless has_residual); must not overlap y
 *             (the kernels write y before they have read all of residual)
 *   y         [n,h',w',c_out] out_dtype
 *   mask_out  d of Section 3.1, one bit per activation: bit (c & 31) of 32-bit word
 *             m*ceil(c_out/32) + (c >> 5), m the pixel row; unused high bits 0.  NULL: not
 *             written.
 *   workspace device scratch of at least cg_conv_workspace_bytes(h) bytes (NULL if that is 0)
 *   cuda_stream  a cudaStream_t (NULL = default stream)
 * Enqueues on the stream and returns without synchronising; back-to-back calls are fine.
 * A NaN partial sum does not fire.  Errors: CG_ERR_INVALID_ARG, CG_ERR_ALIGNMENT (x, weights,
 * y, residual need 16-byte alignment, mask_out 4), CG_ERR_WORKSPACE, CG_ERR_CUDA. */
cg_status cg_conv_forward(cg_conv_t h, const void* x, const void* w_base, const void* w_cond,
                          const cg_bn_params* bn, const float* delta, const void* residual,
                          void* y, uint32_t* mask_out, void* workspace, size_t workspace_bytes,
                          void* cuda_stream);

/* Same layer with x, residual, y and mask_out in HOST memory (pinned memory makes the copies
 * asynchronous).  Weights, bn and delta stay device pointers.  `staging` is device scratch of
 * at least cg_conv_host_staging_bytes(h) bytes that holds x, y, mask and the workspace.
 * Copies in, runs the layer, copies out, all on `cuda_stream`; does not synchronise. */
size_t cg_conv_host_staging_bytes(cg_conv_t h);
cg_status cg_conv_forward_host(cg_conv_t h, const void* x_host, const void* w_base,
                               const void* w_cond, const cg_bn_params* bn, const float* delta,
                               const void* residual_host, void* y_host, uint32_t* mask_host,
                               void* staging, size_t staging_bytes, void* cuda_stream);

/* Base path only (Section 3.1: P = W_p*x_p): writes P as [M,c_out] fp32 (int32 for I8) on the
 * device.  For calibrating gate statistics and thresholds; not on the hot path. */
cg_status cg_conv_partial_sums(cg_conv_t h, const void* x, const void* w_base, void* p_out,
                               void* cuda_stream);

/* Synchronises `cuda_stream`, copies the counters to *out and clears them.  Returns
 * out->device_status if a kernel reported a problem, else CG_OK. */
cg_status cg_conv_stats(cg_conv_t h, cg_stats* out, void* cuda_stream);

/* Number of kernel launches one cg_conv_forward enqueues for this layer. */
int cg_conv_launches_per_forward(cg_conv_t h);

/* 1 if the tensor-core path runs this layer, 0 if the direct path does. */
int cg_conv_uses_tensor_cores(cg_conv_t h);

/* Which kernel family runs this layer (Section 3.1's two convolutions, gate and combine fused
 * in all of them): the CUDA-core direct kernels, the tcgen05 kernel with pixels on the MMA's M
 * side, the tcgen05 kernel with output channels on the M side and pixels on the N side, or the
 * tcgen05 kernel with pixels on the M side and (horizontal tap, output channel) on the N side. */
typedef enum {
  CG_KERNEL_DIRECT = 0,
  CG_KERNEL_TENSOR_PIXEL_MAJOR = 1,
  CG_KERNEL_TENSOR_CHANNEL_MAJOR = 2,
  CG_KERNEL_TENSOR_TAP_STACKED = 3
} cg_kernel_id;
int cg_conv_kernel_id(cg_conv_t h);

/* Writes a one-line description of the tiling chosen for this layer (tile sizes, K stages, ring
 * depth, grid) into buf; returns the length snprintf would have written, -1 on a NULL argument. */
int cg_conv_plan_string(cg_conv_t h, char* buf, size_t len);

void cg_conv_destroy(cg_conv_t h);

/* (No counterpart in the paper: a packaging variant of the same layer.)
 * The gated layer for callers that cannot allocate device memory: code that runs inside a
 * framework or memory pool that owns the whole device, loops that must not make calls which
 * can synchronise the device, plug-ins that are handed tensors but no allocator.  The regular
 * API needs a handle, and cg_conv_create allocates; this call needs no handle and allocates
 * nothing, on the device or through any library.  Its scratch -- the activity counters and the
 * per-channel gate/batch-norm constants that a small prologue kernel folds on every call -- is
 * a fixed array inside the library image, which costs every GPU that loads the library about
 * 40 KB until the process exits.
 *   desc      the layer, as for cg_conv_create (algo and cond_mode are ignored: the CUDA-core
 *             direct kernels run it, so results equal cg_conv_forward with CG_ALGO_DIRECT);
 *             F32 and BF16 only, else CG_ERR_UNSUPPORTED
 *   x .. mask_out   device pointers exactly as for cg_conv_forward
 *   stats_out NULL, or a host struct to fill (outputs, active, dense/gated/executed MACs); a
 *             non-NULL value makes the call synchronise the stream
 * Limit: desc->c_out <= CG_STATIC_MAX_C_OUT, else CG_ERR_WORKSPACE (the constants would not
 * fit the fixed array).  Other errors as cg_conv_forward.
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside any stream capture.
 * Every call on a device uses the same array and overwrites what the previous call left
 * there (the counters are cleared by the prologue), so two calls that can overlap on the GPU
 * -- different streams, or the same stream from two threads -- race; serialise them. */
#define CG_STATIC_MAX_C_OUT 2048
cg_status cg_conv_forward_static(const cg_conv_desc* desc, const void* x, const void* w_base,
                                 const void* w_cond, const cg_bn_params* bn, const float* delta,
                                 const void* residual, void* y, uint32_t* mask_out,
                                 cg_stats* stats_out, void* cuda_stream);

const char* cg_status_string(cg_status s);

#ifdef __cplusplus
}
#endif
#endif /* CGCONV_H_ */
